"""Parity of the CUDA path against the CPU oracle, through the C ABI (ctypes binding).

Structure (pos / crd) must match bit for bit; values within 1e-12 (f64) / 1e-5 (f32) relative
per entry, or within that factor of sum|a*b| where mixed-sign products cancel.
"""
import numpy as np
import pytest

from helpers import TOL, read_hand_case, rows_of, values_close
from workloads import (CSR, CSF3, config_inputs, random_csr, rmat_csr, stencil27_csr, uniform_csf3,
                       uniform_rows_csr)

pytestmark = pytest.mark.gpu

POLICIES = ("dense", "ism", "auto", "hash")
# thresholds that force every route on small inputs
SMALL_ROUTES = dict(ism_warp_cap=8, ism_cta_cap=64, dense_unit_outputs=64, fallback_cap=16)
GLOBAL, DENSE = 7, slice(4, 7)          # indices into stats["rows_per_class"]


@pytest.fixture(scope="module")
def ctx():
    import torch
    from paper_2404_04541_b200 import api
    assert torch.cuda.is_available()
    return api.Context("cuda")


def run_spgemm(ctx, A, B, policy="auto", **options):
    from paper_2404_04541_b200 import api
    dA = api.DeviceCSR.from_host(A)
    dB = dA if B is A else api.DeviceCSR.from_host(B)
    C, stats = ctx.spgemm(dA, dB, policy=policy, **options)
    return C.pos.cpu().numpy(), C.crd.cpu().numpy(), C.val.cpu().numpy(), stats


def assert_matches(got, ref, dtype, rows=None, exact_values=False):
    pos, crd, val = got
    assert np.array_equal(pos, ref.pos), "row pointer differs"
    assert np.array_equal(crd, ref.crd), "column indices differ"
    if exact_values:
        assert np.array_equal(val, ref.val.astype(dtype))
        return 0
    ok, second = values_close(val, ref.val_ref, ref.abs, TOL[np.dtype(dtype)])
    assert ok.all(), f"{(~ok).sum()} of {ok.size} values out of tolerance"
    return second


def check_spgemm(ctx, oracle_mod, A, B, policy="auto", exact_values=False, threads=4, **options):
    ref = oracle_mod.spgemm(A, B, threads=threads)
    pos, crd, val, stats = run_spgemm(ctx, A, B, policy, **options)
    assert stats["products"] == int(ref.products.sum())
    assert stats["nnz"] == ref.nnz
    assert_matches((pos, crd, val), ref, A.val.dtype, exact_values=exact_values)
    return stats


# ------------------------------------------------------------------ hand-worked cases
@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("name", ["hand_dedupe_4x4.txt", "hand_cancel_4x4.txt", "hand_rect_3x5x4.txt"])
def test_hand_cases(ctx, name, policy):
    A, B, cr, cc, cv, products = read_hand_case(name)
    pos, crd, val, stats = run_spgemm(ctx, A, B, policy)
    assert np.array_equal(rows_of(pos), cr) and np.array_equal(crd, cc) and np.array_equal(val, cv)
    assert stats["products"] == products.sum()


# ------------------------------------------------------------------ random small, every route
@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("m,k,n,dens,seed", [(1, 1, 1, 1.0, 0), (37, 64, 700, 0.08, 1), (200, 150, 1000, 0.05, 2),
                                             (64, 64, 64, 0.5, 3), (129, 300, 5000, 0.02, 4)])
def test_random_small_all_routes(ctx, oracle_mod, policy, m, k, n, dens, seed):
    A = random_csr(m, k, dens, seed, empty_row_frac=0.1)
    B = random_csr(k, n, dens, seed + 9, empty_row_frac=0.1)
    check_spgemm(ctx, oracle_mod, A, B, policy)                      # default thresholds
    stats = check_spgemm(ctx, oracle_mod, A, B, policy, **SMALL_ROUTES)
    if policy == "ism" and m >= 37:
        assert stats["rows_per_class"][GLOBAL] > 0                   # the global-memory ISM ran
    if policy == "dense" and n >= 700:                               # rows beyond a warp's capacity went to CTA units
        assert stats["dense_units"] == sum(stats["rows_per_class"][DENSE]) - stats["dense_warp_rows"] > 0


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("policy", POLICIES)
def test_policy_equivalence_and_dtypes(ctx, oracle_mod, policy, dtype):
    A = random_csr(300, 300, 0.03, 5, dtype=dtype, empty_row_frac=0.05)
    check_spgemm(ctx, oracle_mod, A, A, policy, **SMALL_ROUTES)
    check_spgemm(ctx, oracle_mod, A, A, policy)


def _rows_with_products(targets, ncols, seed, dtype=np.float64):
    """A (R x 2R), B (2R x ncols): row r of A*B has exactly targets[r] products, about half of
    them colliding."""
    rng = np.random.default_rng(seed)
    R = len(targets)
    rows, cols, vals = [], [], []
    for r, P in enumerate(targets):
        l0, l1 = (P + 1) // 2, P // 2
        width = min(ncols, max(l0, int(1.5 * l0) + 1))
        lo = int(rng.integers(0, ncols - width + 1))
        for b, ln in ((2 * r, l0), (2 * r + 1, l1)):
            c = np.sort(rng.choice(width, size=ln, replace=False)) + lo
            rows.append(np.full(ln, b)); cols.append(c); vals.append(rng.uniform(-1, 1, ln))
    Bm = CSR.from_coo(2 * R, ncols, np.concatenate(rows), np.concatenate(cols), np.concatenate(vals), dtype=dtype)
    Am = CSR.from_coo(R, 2 * R, np.repeat(np.arange(R), 2), np.arange(2 * R), rng.uniform(-1, 1, 2 * R), dtype=dtype)
    return Am, Bm


@pytest.mark.parametrize("policy", POLICIES)
def test_capacity_boundaries(ctx, oracle_mod, policy):
    targets = [1, 2, 7, 8, 9, 15, 16, 17, 31, 32, 33, 63, 64, 65, 255, 256, 257, 511, 512, 513, 1023, 1024, 1025,
               4095, 4096, 4097, 8191, 8192, 8193, 20000]
    A, B = _rows_with_products(targets, 40000, 11)
    stats = check_spgemm(ctx, oracle_mod, A, B, policy)
    assert stats["max_row_products"] == 20000
    if policy in ("ism", "hash"):
        assert stats["rows_per_class"][GLOBAL] == 5                  # rows above the shared-memory capacity
    if policy == "hash":                                             # the two table sizes split at 1024 products
        assert stats["rows_per_class"][8] == 22 and stats["rows_per_class"][9] == 3
    A, B = _rows_with_products(targets[:17], 3000, 12)
    check_spgemm(ctx, oracle_mod, A, B, policy, **SMALL_ROUTES)


@pytest.mark.parametrize("policy", POLICIES)
def test_edge_cases(ctx, oracle_mod, policy):
    # all-empty A, empty B rows, one huge row among empty ones
    z = np.zeros(0)
    A0 = CSR.from_coo(5, 6, z, z, z)
    B0 = random_csr(6, 9, 0.5, 1)
    check_spgemm(ctx, oracle_mod, A0, B0, policy)
    A1 = random_csr(20, 30, 0.3, 2)
    B1 = CSR.from_coo(30, 40, z, z, z)
    check_spgemm(ctx, oracle_mod, A1, B1, policy)
    rng = np.random.default_rng(3)
    cols = np.sort(rng.choice(3000, 2000, replace=False))
    A2 = CSR.from_coo(50, 3000, np.full(2000, 17), cols, rng.uniform(-1, 1, 2000))
    B2 = uniform_rows_csr(3000, 5000, 40, 4)
    stats = check_spgemm(ctx, oracle_mod, A2, B2, policy)
    assert stats["max_row_products"] == 80000 and stats["rows_per_class"][0] == 49
    # many A entries that pick empty B rows: a row with few products but a long A row
    live = np.nonzero(rng.random(3000) < 0.01)[0]
    B3 = CSR.from_coo(3000, 5000, np.repeat(live, 5),
                      np.concatenate([np.sort(rng.choice(5000, 5, replace=False)) for _ in live]),
                      rng.uniform(-1, 1, 5 * live.size))
    check_spgemm(ctx, oracle_mod, A2, B3, policy)


@pytest.mark.parametrize("policy", ["dense", "auto"])
def test_heavy_row_is_split_over_several_units(ctx, oracle_mod, policy):
    """A row with ~400 k products is shared by several CTAs (each takes a slice of its A entries
    and adds into the same outputs); with a 64-output shared-memory accumulator most outputs
    accumulate in global memory."""
    rng = np.random.default_rng(5)
    cols = np.sort(rng.choice(4000, 2000, replace=False))
    A = CSR.from_coo(40, 4000, np.concatenate([np.full(2000, 7), np.arange(40)]),
                     np.concatenate([cols, rng.integers(0, 4000, 40)]), rng.uniform(-1, 1, 2040))
    A = CSR.from_dense(A.to_dense())                                 # merges accidental duplicates
    B = uniform_rows_csr(4000, 30000, 200, 6)
    for opts in ({}, dict(dense_unit_outputs=64)):
        stats = check_spgemm(ctx, oracle_mod, A, B, policy, **opts)
        assert stats["max_row_products"] >= 400000
        assert stats["dense_units"] >= sum(stats["rows_per_class"][DENSE]) - stats["dense_warp_rows"] + 3


def test_ism_routes_reproduce_sequential_sum(ctx, oracle_mod):
    """The register and shared-memory ISM routes add each row's products in loop order with a
    separate multiply and add, so they give the oracle's plain double-precision sum bit for bit.
    (The global-memory route reduces each accumulation-array round before merging it, which
    re-associates the sum, so it is only held to the tolerance.)"""
    A = random_csr(200, 200, 0.04, 8)
    ref = oracle_mod.spgemm(A, A)
    for opts in ({}, dict(ism_warp_cap=8, ism_cta_cap=1024), dict(ism_warp_cap=16, ism_cta_cap=256)):
        pos, crd, val, stats = run_spgemm(ctx, A, A, "ism", **opts)
        assert stats["rows_per_class"][GLOBAL] == 0
        assert np.array_equal(pos, ref.pos) and np.array_equal(crd, ref.crd)
        assert (val != ref.val).sum() == 0


def test_warp_dense_route_reproduces_sequential_sum(ctx, oracle_mod):
    """With its lanes across one B row at a time, the warp-per-row dense workspace sums every
    output in loop order.  That holds for rows whose B rows are long enough for a full-warp
    group (here: the interior grid points, 27 x 27 products); rows with short B rows keep
    several A entries in flight and are held to the tolerance."""
    A = stencil27_csr(10, 3)
    ref = oracle_mod.spgemm(A, A)
    pos, crd, val, stats = run_spgemm(ctx, A, A, "dense")
    assert stats["dense_warp_rows"] == A.nrows
    assert np.array_equal(pos, ref.pos) and np.array_equal(crd, ref.crd)
    interior = np.repeat(ref.products == 729, np.diff(ref.pos))
    assert interior.sum() == 6 ** 3 * 125
    assert np.array_equal(val[interior], ref.val[interior])
    ok, _ = values_close(val, ref.val_ref, ref.abs, 1e-12)
    assert ok.all()


def test_warp_dense_route_compact_and_full_bitmaps(ctx, oracle_mod):
    """The warp dense route saves a row's bitmap either whole or as its non-empty words only.
    One matrix makes rows of every kind under the forced dense policy: a few products over a wide
    span (compact form), many products over a narrow span (whole bitmap: the list would not fit
    the slot), more than 256 outputs (handed to the CTA numeric kernel, which reads the whole
    bitmap), and empty rows."""
    rng = np.random.default_rng(11)
    n = 20000
    B = uniform_rows_csr(n, n, 6, 5)
    rows, cols = [], []
    for i in range(96):
        kind = i % 4
        if kind == 0:
            ks = rng.choice(n, size=3, replace=False)           # 18 products anywhere in 20000 columns
        elif kind == 1:
            ks = rng.choice(n, size=30, replace=False)          # 180 products, still sparse words
        elif kind == 2:
            ks = rng.choice(n, size=120, replace=False)         # ~700 outputs: beyond a warp's accumulator
        else:
            ks = np.array([], dtype=np.int64)
        rows += [i] * len(ks)
        cols += sorted(int(k) for k in ks)
    A = CSR.from_coo(96, n, rows, cols, rng.uniform(-1, 1, len(rows)))
    # a block of rows that all pick B rows with the same few columns: narrow span, dense words
    Bn = CSR.from_coo(64, 40, np.repeat(np.arange(64), 20), np.tile(np.arange(0, 40, 2), 64), rng.uniform(-1, 1, 64 * 20))
    An = uniform_rows_csr(50, 64, 9, 6)
    for (X, Y) in ((A, B), (An, Bn)):
        stats = check_spgemm(ctx, oracle_mod, X, Y, "dense")
        assert stats["rows_per_class"][4] > 0
    # the wide case must have used both numeric kernels
    stats = check_spgemm(ctx, oracle_mod, A, B, "dense")
    assert 0 < stats["dense_warp_rows"] < 72 and stats["dense_units"] > 0


@pytest.mark.parametrize("summaries", [True, False])
@pytest.mark.parametrize("per_row", [1, 2, 5, 10, 20])
def test_bounds_kernel_widths_with_and_without_b_row_summaries(ctx, oracle_mod, per_row, summaries):
    """The bounds kernel gives a row 1, 2, 4, 8 or 32 lanes by A's mean row length, and reads per-B-row
    summaries (first / last column, length) when A has at least four entries per B row, else B's own
    arrays: every combination against the oracle, B with empty rows."""
    m = 3000
    k = 500 if summaries else 40000
    assert (m * per_row >= 4 * k) == summaries
    A = uniform_rows_csr(m, k, per_row, 11 + per_row)
    B = random_csr(k, 6000, 0.002, 12 + per_row, empty_row_frac=0.25)
    for policy in ("auto", "dense"):
        check_spgemm(ctx, oracle_mod, A, B, policy)


@pytest.mark.parametrize("summaries", [True, False])
def test_bounds_of_rows_with_thousands_of_entries(ctx, oracle_mod, summaries):
    """Rows of A with more than 1024 entries get a CTA each in the bounds pass (listed by the lane-group
    kernel, which skips them): a few such rows of different lengths among short and empty ones, at the
    1024 / 1025 edge too, B with empty rows, with the per-B-row summaries and without."""
    k = 7000
    rng = np.random.default_rng(5)
    lengths = [0, 3, 1024, 1025, 0, 6999, 17, 2500, 1, 4097] + [int(x) for x in rng.integers(0, 40, 300)]
    rows, cols = [], []
    for i, n in enumerate(lengths):
        rows.append(np.full(n, i))
        cols.append(np.sort(rng.choice(k, n, replace=False)))
    rows, cols = np.concatenate(rows), np.concatenate(cols)
    A = CSR.from_coo(len(lengths), k, rows, cols, rng.uniform(-1, 1, rows.size))
    if summaries:                                   # at least four A entries per B row: stack A on itself
        reps = 4 * k // A.nnz + 1
        A = CSR.from_coo(reps * len(lengths), k, np.concatenate([rows + r * len(lengths) for r in range(reps)]),
                         np.tile(cols, reps), rng.uniform(-1, 1, reps * rows.size))
    assert (A.nnz >= 4 * k) == summaries
    B = random_csr(k, 3000, 0.003, 6, empty_row_frac=0.3)
    for policy in ("auto", "dense"):
        stats = check_spgemm(ctx, oracle_mod, A, B, policy)
        assert stats["rows"] == A.nrows


@pytest.mark.parametrize("seed", [1, 2, 3])
def test_randomized_shapes_policies_and_thresholds(ctx, oracle_mod, seed):
    """Seeded random sweep: shapes from 1 x 1 to a few thousand rows and up to 2^20 columns, uniform /
    power-law / stencil / heavy-row structure, both value types, every policy, and route thresholds
    drawn at random, each case against the oracle (structure exact, values within the tolerance)."""
    rng = np.random.default_rng(seed)
    for _ in range(16):
        kind = int(rng.integers(0, 5))
        dtype = np.float64 if rng.random() < 0.7 else np.float32
        s = int(rng.integers(1, 1 << 30))
        if kind == 0:
            m, k, n = int(rng.integers(1, 400)), int(rng.integers(1, 400)), int(rng.integers(1, 70000))
            A = random_csr(m, k, float(rng.uniform(0.01, 0.5)), s, empty_row_frac=float(rng.uniform(0, 0.3)))
            B = random_csr(k, n, float(rng.uniform(0.0005, 0.05)), s + 1, empty_row_frac=float(rng.uniform(0, 0.3)))
        elif kind == 1:
            A = B = rmat_csr(int(rng.integers(6, 13)), int(rng.integers(2, 24)), s)
        elif kind == 2:
            A = B = stencil27_csr(int(rng.integers(3, 13)), s)
        elif kind == 3:
            m, k = int(rng.integers(1, 3000)), int(rng.integers(1, 5000))
            A = uniform_rows_csr(m, k, int(rng.integers(1, min(k, 40) + 1)), s)
            n = int(rng.integers(64, 1 << 20))
            B = uniform_rows_csr(k, n, int(rng.integers(1, min(n, 64) + 1)), s + 1)
        else:                                       # a few very heavy rows over a wide span
            k, n = int(rng.integers(500, 3000)), int(rng.integers(20000, 400000))
            B = uniform_rows_csr(k, n, int(rng.integers(20, 200)), s + 1)
            A = random_csr(int(rng.integers(2, 30)), k, float(rng.uniform(0.2, 1.0)), s)
        A.val = A.val.astype(dtype)
        B.val = B.val.astype(dtype)
        policy = POLICIES[int(rng.integers(0, 4))]
        if policy in ("ism", "hash") and kind in (1, 4):
            policy = "auto"                         # the global-memory ISM on very heavy rows is slow
        opts = {}
        if rng.random() < 0.5:
            opts = dict(ism_warp_cap=int(rng.choice([4, 8, 16, 32])), ism_cta_cap=int(rng.choice([64, 256, 1024, 4096])),
                        dense_unit_outputs=int(rng.choice([64, 256, 4096])), fallback_cap=int(rng.choice([2, 16, 256, 2048])))
        if policy == "dense" and B.ncols > (1 << 19):
            # a row may be wider than the widest dense workspace: the forced policy must then say so
            from paper_2404_04541_b200 import binding
            try:
                check_spgemm(ctx, oracle_mod, A, B, policy, **opts)
            except binding.SpwsError as e:
                assert e.status == binding.SPWS_WORKSPACE_TOO_LARGE
        else:
            check_spgemm(ctx, oracle_mod, A, B, policy, **opts)


def test_hash_workspace_load_factor_and_duplicates(ctx, oracle_mod):
    """Rows at the hash workspace's limits: as many DISTINCT columns as a table may take (1024 and
    4096 products, no two colliding: half-full tables), one product more (next table / next route),
    and rows whose products nearly all fall on a few columns (long probe-free chains of adds)."""
    rng = np.random.default_rng(17)
    ncols = 1 << 20
    rows, cols, arow, acol = [], [], [], []
    for r, P in enumerate([1023, 1024, 1025, 4095, 4096, 4097]):
        c = np.sort(rng.choice(ncols, size=P, replace=False))       # one B row per output row: all distinct
        rows.append(np.full(P, r)); cols.append(c); arow.append(r); acol.append(r)
    # rows 6..9: 64 B rows that all hold the same 50 columns -> 3200 products on 50 outputs
    same = np.sort(rng.choice(ncols, size=50, replace=False))
    for b in range(6, 70):
        rows.append(np.full(50, b)); cols.append(same)
    for r in range(6, 10):
        arow += [r] * 64; acol += list(range(6, 70))
    B = CSR.from_coo(70, ncols, np.concatenate(rows), np.concatenate(cols), rng.uniform(-1, 1, sum(len(c) for c in cols)))
    A = CSR.from_coo(10, 70, arow, acol, rng.uniform(-1, 1, len(arow)))
    stats = check_spgemm(ctx, oracle_mod, A, B, "hash")
    assert stats["rows_per_class"][8] == 2 and stats["rows_per_class"][9] == 7 and stats["rows_per_class"][GLOBAL] == 1
    assert stats["nnz"] == 1023 + 1024 + 1025 + 4095 + 4096 + 4097 + 4 * 50


# ------------------------------------------------------------------ benchmark configurations
@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("cfg", ["uniform8", "rmat18", "stencil64"])
def test_reduced_configs(ctx, oracle_mod, cfg, policy):
    c = config_inputs(cfg, reduced=True)
    check_spgemm(ctx, oracle_mod, c["A"], c["B"], policy)


@pytest.mark.parametrize("policy", ["ism", "auto"])
def test_wide_reduced(ctx, oracle_mod, policy):
    c = config_inputs("wide26", reduced=True)
    check_spgemm(ctx, oracle_mod, c["A"], c["B"], policy)


@pytest.mark.parametrize("policy", ["ism", "auto"])
def test_wide_columns_with_many_products(ctx, oracle_mod, policy):
    """2^26 columns and rows with hundreds to thousands of products: the shared-memory ISM must
    sort 64-bit (column, slot) words here (26 column bits + 12 slot bits do not fit 32)."""
    B = uniform_rows_csr(300, 1 << 26, 24, 21)
    A = random_csr(80, 300, 0.12, 22, empty_row_frac=0.1)
    A.val[:] = np.round(A.val * 16) / 16
    stats = check_spgemm(ctx, oracle_mod, A, B, policy)
    assert stats["rows_per_class"][2] + stats["rows_per_class"][3] > 0
    Abig = random_csr(12, 300, 0.6, 23)                               # ~4300 products per row -> beyond 4096
    check_spgemm(ctx, oracle_mod, Abig, B, policy)


def test_dense_cta_widest_span_and_just_beyond(ctx, oracle_mod):
    """Rows whose outputs cover almost 2^19 columns (the widest dense workspace one CTA holds, with
    the whole bitmap and its ranks in shared memory) and rows a little wider, which must fall back
    to the insert-sort-merge workspace in global memory."""
    ncols = 600_000
    B = uniform_rows_csr(96, ncols, 128, 31)
    crd, pos = B.crd, B.pos
    # rows 0..63 of B are clipped to the first 2^19 columns; rows 64..95 keep all 600 000
    out_pos, out_crd, out_val = [0], [], []
    for k in range(B.nrows):
        c = crd[pos[k]:pos[k + 1]]
        v = B.val[pos[k]:pos[k + 1]]
        if k < 64:
            sel = c < (1 << 19)
            c, v = c[sel], v[sel]
        out_crd.append(c); out_val.append(v); out_pos.append(out_pos[-1] + c.size)
    Bc = CSR(B.nrows, ncols, np.asarray(out_pos, dtype=np.int64), np.concatenate(out_crd).astype(np.int32),
             np.concatenate(out_val))
    Bc.val[:] = np.round(Bc.val * 16) / 16
    a_pos = np.array([0, 64, 160], dtype=np.int64)                     # row 0: narrow B rows, row 1: all B rows
    a_crd = np.concatenate([np.arange(64), np.arange(96)]).astype(np.int32)
    a_val = (1 + (np.arange(160) % 7) / 8.0).astype(np.float64)
    A = CSR(2, 96, a_pos, a_crd, a_val)
    stats = check_spgemm(ctx, oracle_mod, A, Bc, "auto")
    assert sum(stats["rows_per_class"][DENSE]) == 1 and stats["rows_per_class"][GLOBAL] == 1


def test_dense_policy_refuses_prohibitive_workspace(ctx):
    from paper_2404_04541_b200 import binding
    c = config_inputs("wide26", reduced=True)
    with pytest.raises(binding.SpwsError) as e:
        run_spgemm(ctx, c["A"], c["B"], "dense")
    assert e.value.status == binding.SPWS_WORKSPACE_TOO_LARGE


def test_full_uniform8(ctx, oracle_mod):
    c = config_inputs("uniform8")
    stats = check_spgemm(ctx, oracle_mod, c["A"], c["B"], "auto")
    assert stats["products"] == 131072


def test_full_stencil64(ctx, oracle_mod):
    """Values in [0.5, 1.5] cannot cancel, so every entry must pass the plain relative clause."""
    c = config_inputs("stencil64")
    A = c["A"]
    ref = oracle_mod.spgemm(A, A, threads=oracle_mod.hardware_threads())
    pos, crd, val, stats = run_spgemm(ctx, A, A, "auto")
    assert stats["products"] == 566 ** 3 and stats["nnz"] == 314 ** 3 == ref.nnz
    second = assert_matches((pos, crd, val), ref, np.float64)
    assert second == 0


def test_full_wide26(ctx, oracle_mod):
    c = config_inputs("wide26")
    A, B = c["A"], c["B"]
    ref = oracle_mod.spgemm(A, B, threads=4)
    pos, crd, val, stats = run_spgemm(ctx, A, B, "auto")
    assert stats["rows_per_class"][1] == A.nrows                     # register ISM for every row
    second = assert_matches((pos, crd, val), ref, np.float32)
    single = np.repeat(ref.products == np.diff(ref.pos), np.diff(ref.pos))   # rows without any collision
    assert np.array_equal(val[single], ref.val[single].astype(np.float32))   # one correctly rounded multiply
    assert second <= ref.nnz - single.sum()


def test_full_rmat18_sampled_rows_and_invariants(ctx, oracle_mod):
    """Full-size power-law config in the launch configuration the benchmark times: the row
    pointer is checked against properties that hold at any size, and sampled rows (the heaviest
    ones included) against the oracle entry by entry."""
    import torch
    from paper_2404_04541_b200 import api
    c = config_inputs("rmat18")
    A = c["A"]
    dA = api.DeviceCSR.from_host(A)
    C, stats = ctx.spgemm(dA, dA, policy="auto")
    lens = np.diff(A.pos)
    ub = np.bincount(rows_of(A.pos), weights=lens[A.crd], minlength=A.nrows).astype(np.int64)
    assert stats["products"] == ub.sum()
    pos = C.pos.cpu().numpy()
    cnt = np.diff(pos)
    assert pos[0] == 0 and pos[-1] == stats["nnz"] == C.crd.shape[0]
    assert (cnt <= np.minimum(ub, A.ncols)).all() and ((cnt == 0) == (ub == 0)).all()
    # sorted and unique inside every row (checked on the device)
    crd = C.crd
    inc = torch.ones(crd.shape[0], dtype=torch.bool, device=crd.device)
    inc[1:] = crd[1:] > crd[:-1]
    starts = C.pos[:-1][torch.from_numpy(cnt > 0).to(crd.device)]
    inc[starts] = True
    assert bool(inc.all())
    # C*1 = A*(B*1)
    b1 = np.bincount(rows_of(A.pos), weights=A.val, minlength=A.nrows)
    ab1 = np.bincount(rows_of(A.pos), weights=A.val * b1[A.crd], minlength=A.nrows)
    absb1 = np.bincount(rows_of(A.pos), weights=np.abs(A.val), minlength=A.nrows)
    scale = np.bincount(rows_of(A.pos), weights=np.abs(A.val) * absb1[A.crd], minlength=A.nrows)
    rowid = torch.repeat_interleave(torch.arange(A.nrows, device=crd.device), torch.from_numpy(cnt).to(crd.device))
    c1 = torch.zeros(A.nrows, dtype=torch.float64, device=crd.device).index_add_(0, rowid, C.val).cpu().numpy()
    assert (np.abs(c1 - ab1) <= 1e-12 * scale + 1e-300).all()
    # sampled rows against the oracle: the 3 heaviest, 3 around each class boundary, 300 random
    order = np.argsort(ub)
    rng = np.random.default_rng(0)
    pick = set(order[-3:].tolist()) | set(rng.choice(A.nrows, 300, replace=False).tolist())
    for edge in (32, 256, 4096):
        near = np.argsort(np.abs(ub - edge))[:3]
        pick |= set(near.tolist())
    rows = np.array(sorted(pick))
    ref = oracle_mod.spgemm(A, A, rows=rows, threads=oracle_mod.hardware_threads())
    crd_h = None
    for t, r in enumerate(rows):
        s, e = int(pos[r]), int(pos[r + 1])
        assert e - s == ref.pos[t + 1] - ref.pos[t]
        got_c = C.crd[s:e].cpu().numpy()
        got_v = C.val[s:e].cpu().numpy()
        u = slice(ref.pos[t], ref.pos[t + 1])
        assert np.array_equal(got_c, ref.crd[u])
        ok, _ = values_close(got_v, ref.val_ref[u], ref.abs[u], 1e-12)
        assert ok.all()


def test_full_rmat18_every_entry_streamed(ctx, oracle_mod):
    """The whole power-law result against the oracle, entry by entry, in the launch configuration
    the benchmark times.  Both sides are walked in blocks of rows so that neither 15 GB result has
    to sit in host memory: the oracle computes a block, the matching slices of C come off the
    device, structure must be identical and every value must pass the two-clause rule."""
    from paper_2404_04541_b200 import api
    c = config_inputs("rmat18")
    A = c["A"]
    dA = api.DeviceCSR.from_host(A)
    C, stats = ctx.spgemm(dA, dA, policy="auto")
    pos = C.pos.cpu().numpy()
    threads = oracle_mod.hardware_threads()
    # blocks of about 2^24 products (row boundaries), so that each oracle call stays small
    lens = np.diff(A.pos)
    ub = np.bincount(rows_of(A.pos), weights=lens[A.crd], minlength=A.nrows).astype(np.int64)
    csum = np.concatenate([[0], np.cumsum(ub)])
    cuts = np.unique(np.searchsorted(csum, np.arange(0, csum[-1], 1 << 25)))
    cuts = np.unique(np.concatenate([cuts, [0, A.nrows]]))
    products = entries = second = 0
    for r0, r1 in zip(cuts[:-1], cuts[1:]):
        ref = oracle_mod.spgemm(A, A, rows=np.arange(r0, r1), threads=threads)
        s, e = int(pos[r0]), int(pos[r1])
        assert np.array_equal(pos[r0:r1 + 1] - s, ref.pos), f"row pointer differs in rows {r0}..{r1}"
        assert np.array_equal(C.crd[s:e].cpu().numpy(), ref.crd), f"column indices differ in rows {r0}..{r1}"
        ok, sec = values_close(C.val[s:e].cpu().numpy(), ref.val_ref, ref.abs, 1e-12)
        assert ok.all(), f"{(~ok).sum()} values out of tolerance in rows {r0}..{r1}"
        products += int(ref.products.sum())
        entries += ref.nnz
        second += sec
    assert products == stats["products"] and entries == stats["nnz"] == int(pos[-1])
    print(f"rmat18: {entries} entries compared, {second} needed the sum|a*b| clause")


# ------------------------------------------------------------------ outer-product form, second-order workspace
def run_outer(ctx, A, B, policy="auto", **options):
    """A is the I x K operand; the library takes it by its rows k, i.e. the CSR of its transpose."""
    from paper_2404_04541_b200 import api
    dAt = api.DeviceCSR.from_host(A.transpose())
    dB = api.DeviceCSR.from_host(B)
    C, stats = ctx.spgemm_outer(dAt, dB, policy=policy, **options)
    return C.pos.cpu().numpy(), C.crd.cpu().numpy(), C.val.cpu().numpy(), stats


@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("m,k,n,dens,seed", [(1, 1, 1, 1.0, 0), (37, 64, 700, 0.08, 1), (200, 150, 1000, 0.05, 2),
                                             (64, 64, 64, 0.5, 3), (300, 20, 5000, 0.1, 4)])
def test_outer_product_matches_the_rowwise_oracle(ctx, oracle_mod, policy, m, k, n, dens, seed):
    A = random_csr(m, k, dens, seed, empty_row_frac=0.1)
    B = random_csr(k, n, dens, seed + 9, empty_row_frac=0.1)
    ref = oracle_mod.spgemm(A, B)
    pos, crd, val, stats = run_outer(ctx, A, B, policy)
    assert stats["products"] == int(ref.products.sum()) and stats["nnz"] == ref.nnz
    assert_matches((pos, crd, val), ref, np.float64)


@pytest.mark.parametrize("dtype", [np.float32, np.float64])
@pytest.mark.parametrize("cap", [0, 1, 2, 3, 7, 1000, 10 ** 6])
def test_outer_product_sparse_workspace_reproduces_algorithm1(ctx, oracle_mod, cap, dtype):
    """The sparse second-order workspace with an accumulation array of `cap` components sums in the
    order Algorithm 1 fixes (sort and reduce the full array on its own, then all + accumulated), so
    with separate multiply and add it must equal the oracle's restatement bit for bit (f64) at
    every capacity; one round (cap 0) equals the plain loop-order sum k -> i -> j."""
    A = random_csr(60, 50, 0.15, 21, empty_row_frac=0.1)
    B = random_csr(50, 90, 0.15, 22, empty_row_frac=0.1)
    A.val = A.val.astype(dtype)
    B.val = B.val.astype(dtype)
    P = int(oracle_mod.spgemm(A, B).products.sum())
    ref = oracle_mod.ism_outer(A, B, cap if cap > 0 else P)
    pos, crd, val, stats = run_outer(ctx, A, B, "ism", outer_cap=cap)
    assert np.array_equal(pos, ref.pos) and np.array_equal(crd, ref.crd)
    if dtype == np.float64:
        assert np.array_equal(val, ref.val)
    else:
        assert np.allclose(val, ref.val, rtol=1e-5, atol=1e-6)


def test_outer_product_on_a_power_law_matrix_and_wide_labels(ctx, oracle_mod):
    A = rmat_csr(11, 8, 5)
    ref = oracle_mod.spgemm(A, A, threads=4)
    for policy in POLICIES:
        pos, crd, val, stats = run_outer(ctx, A, A, policy)
        assert_matches((pos, crd, val), ref, np.float64)
    # labels beyond 32 bits: 3000 x 2^22 outputs; the dense workspace cannot be offered here
    B = uniform_rows_csr(500, 1 << 22, 6, 7)
    A2 = random_csr(3000, 500, 0.01, 8)
    ref = oracle_mod.spgemm(A2, B)
    pos, crd, val, stats = run_outer(ctx, A2, B, "auto")
    assert stats["rows_per_class"][GLOBAL] == 3000
    assert_matches((pos, crd, val), ref, np.float64)
    # the dense workspace forced with a scratch buffer that cannot hold I x J values: refused, like
    # the paper's dense workspace running out of memory
    import torch
    from paper_2404_04541_b200 import api, binding
    dAt, dB = api.DeviceCSR.from_host(A2.transpose()), api.DeviceCSR.from_host(B)
    sparse_plan = ctx.plan(api.EXPR_OUTER, (binding.SPWS_CSR,) * 3, np.float64, "ism")
    nbytes = sparse_plan.workspace_size(dAt.arrays(), dB.arrays())
    sparse_plan.close()
    dense_plan = ctx.plan(api.EXPR_OUTER, (binding.SPWS_CSR,) * 3, np.float64, "dense")
    assert dense_plan.workspace_size(dAt.arrays(), dB.arrays()) > 3000 * (1 << 22) * 8
    sc = ctx.scratch(nbytes)
    c = binding.csr_arrays(3000, 1 << 22, torch.empty(3001, dtype=torch.int64, device="cuda"), None, None)
    with pytest.raises(binding.SpwsError) as e:
        dense_plan.symbolic(dAt.arrays(), dB.arrays(), c, ctx._aligned_ptr(sc), nbytes)
    assert e.value.status == binding.SPWS_WORKSPACE_TOO_LARGE
    dense_plan.close()


# ------------------------------------------------------------------ higher-order scatters, COO result
@pytest.mark.parametrize("dims,nnz,L,seed", [((6, 7, 8), 80, 9, 1), ((40, 30, 50), 3000, 64, 2), ((8, 200, 300), 5000, 1000, 3)])
def test_higher_order_scatters_match_the_oracle(ctx, oracle_mod, dims, nnz, L, seed):
    """SpTTM with the outermost mode contracted, SpTTM-I and SpMTTKRP (sparse result in coordinate
    form) against the map oracle: coordinates exact and in lexicographic order, values under the
    two-clause rule, in one round and with accumulation arrays that fill several times."""
    from paper_2404_04541_b200 import api
    B = uniform_csf3(dims, nnz, seed)
    dB = api.DeviceCSF3.from_host(B)
    cases = [
        (api.EXPR_SPTTM, oracle_mod.spttm, [random_csr(dims[0], L, 0.3, seed + 10, empty_row_frac=0.2)]),
        (api.EXPR_SPTTM_I, oracle_mod.spttm_i, [random_csr(dims[1], L, 0.05 if L > 500 else 0.3, seed + 11, empty_row_frac=0.2)]),
        (api.EXPR_SPMTTKRP, oracle_mod.spmttkrp, [random_csr(dims[0], L, 0.3, seed + 12), random_csr(dims[1], L, 0.05 if L > 500 else 0.3, seed + 13)]),
    ]
    for expr, fn, mats in cases:
        ref = fn(B, *mats)
        dm = [api.DeviceCSR.from_host(m) for m in mats]
        caps = [0, max(7, ref.products // 3 + 1)] + ([5] if nnz < 100 else [])
        for cap in caps:
            crd, val, stats = ctx.scatter_coo(expr, dB, *dm, policy="ism", outer_cap=cap)
            assert stats["nnz"] == ref.nnz, expr
            if expr != api.EXPR_SPMTTKRP:
                assert stats["products"] == ref.products, expr     # (SpMTTKRP numbers the C-row elements; some are absent)
            assert np.array_equal(crd.cpu().numpy().astype(np.int64), ref.crd), expr
            ok, _ = values_close(val.cpu().numpy(), ref.val_ref, ref.abs, 1e-12)
            assert ok.all(), expr


def test_higher_order_scatters_refuse_a_dense_workspace(ctx):
    from paper_2404_04541_b200 import api, binding
    with pytest.raises(binding.SpwsError) as e:
        ctx.plan(api.EXPR_SPTTM, (binding.SPWS_COO, binding.SPWS_CSF3, binding.SPWS_CSR), np.float64, "dense")
    assert e.value.status == binding.SPWS_WORKSPACE_TOO_LARGE


# ------------------------------------------------------------------ gather-only lower bound
@pytest.mark.parametrize("name", ["rmat", "stencil", "heavy"])
def test_gather_ceiling_visits_every_product_once(ctx, name):
    """The iteration-only form of the dense numeric kernels must walk exactly the products of the
    rows routed to the dense workspace: with the dense policy forced that is every product, so the
    sum of the gathered column indices (exact) and of the products a*b (to rounding) have closed
    forms in the operands."""
    from paper_2404_04541_b200 import api, binding
    if name == "rmat":
        A = B = rmat_csr(12, 16, 3)
    elif name == "stencil":
        A = B = stencil27_csr(12, 4)
    else:
        B = uniform_rows_csr(4000, 30000, 200, 6)
        A = random_csr(40, 4000, 0.3, 5)
    dA = api.DeviceCSR.from_host(A)
    dB = dA if B is A else api.DeviceCSR.from_host(B)
    plan = ctx.plan(api.EXPR_SPGEMM, (binding.SPWS_CSR,) * 3, np.float64, "dense")
    c, state = ctx.spgemm_symbolic(plan, dA, dB)
    for _ in range(2):                                               # repeatable: the call clears its own counters
        idx_sum, val_sum = ctx.gather_ceiling(plan, c, state)
        col_sum = np.bincount(rows_of(B.pos), weights=B.crd.astype(np.float64), minlength=B.nrows).astype(np.int64)
        assert idx_sum == int(col_sum[A.crd].sum())
        b1 = np.bincount(rows_of(B.pos), weights=B.val, minlength=B.nrows)
        babs = np.bincount(rows_of(B.pos), weights=np.abs(B.val), minlength=B.nrows)
        want, scale = float((A.val * b1[A.crd]).sum()), float((np.abs(A.val) * babs[A.crd]).sum())
        assert abs(val_sum - want) <= 1e-12 * scale
    stats = plan.get_stats()
    assert stats["dense_units"] + stats["dense_warp_rows"] > 0
    plan.close()


# ------------------------------------------------------------------ row-sharded driver on the device
def _sharded_worker(rank, world, port, out_dir):
    import os
    import sys
    sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))
    import torch
    import torch.distributed as dist
    from paper_2404_04541_b200 import api
    from paper_2404_04541_b200 import dist as spd
    from workloads import rmat_csr
    torch.cuda.set_device(0)                        # every rank on the one device: ranks share nothing on the data path
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    A = rmat_csr(11, 12, 9)
    ctx = api.Context("cuda:0")
    res = spd.spgemm_sharded(A, A, spd.local_spgemm_cuda(ctx), spd.row_products_cuda(ctx))
    pos, crd, val = spd.gather_full(res, A.nrows)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), pos=pos, crd=crd, val=val, r0=res.row_begin, r1=res.row_end)
    dist.destroy_process_group()


@pytest.mark.parametrize("world", [1, 2])
def test_sharded_driver_with_the_cuda_local_product(oracle_mod, tmp_path, world):
    """The row-sharded driver with the CUDA path as the local product (upload of a row block,
    symbolic + numeric, row-pointer offsets from the size exchange) against the unsharded oracle."""
    import socket
    import torch.multiprocessing as mp
    with socket.socket() as sk:
        sk.bind(("127.0.0.1", 0))
        port = sk.getsockname()[1]
    mp.spawn(_sharded_worker, args=(world, port, str(tmp_path)), nprocs=world, join=True)
    A = rmat_csr(11, 12, 9)
    ref = oracle_mod.spgemm(A, A)
    for r in range(world):
        o = np.load(str(tmp_path / f"rank{r}.npz"))
        assert np.array_equal(o["pos"], ref.pos) and np.array_equal(o["crd"], ref.crd)
        ok, _ = values_close(o["val"], ref.val_ref, ref.abs, 1e-12)
        assert ok.all()
    if world == 2:
        a, b = (np.load(str(tmp_path / f"rank{r}.npz")) for r in range(2))
        assert a["r0"] == 0 and a["r1"] == b["r0"] and b["r1"] == A.nrows


# ------------------------------------------------------------------ TTM
def run_ttm(ctx, A, B, policy="auto", **options):
    from paper_2404_04541_b200 import api
    C, stats = ctx.ttm(api.DeviceCSF3.from_host(A), api.DeviceCSR.from_host(B), policy=policy, **options)
    f = lambda t: t.cpu().numpy()
    return dict(pos0=f(C.pos0), crd0=f(C.crd0), pos1=f(C.pos1), crd1=f(C.crd1), pos2=f(C.pos2), crd2=f(C.crd2),
                val=f(C.val)), stats


def check_ttm(ctx, oracle_mod, A, B, policy="auto", **options):
    ref = oracle_mod.ttm(A, B)
    got, stats = run_ttm(ctx, A, B, policy, **options)
    for name in ("pos0", "crd0", "pos1", "crd1", "pos2", "crd2"):
        assert np.array_equal(got[name], getattr(ref, name)), name
    ok, _ = values_close(got["val"], ref.val_ref, ref.abs, TOL[np.dtype(A.val.dtype)])
    assert ok.all()
    assert stats["products"] == ref.products.sum()
    return stats


@pytest.mark.parametrize("policy", POLICIES)
def test_ttm_small_and_empty_fibres(ctx, oracle_mod, policy):
    A = CSF3.from_coo((3, 3, 4), [0, 0, 1, 1, 2], [0, 2, 0, 1, 1], [1, 0, 1, 2, 3], [1.0, 2.0, 3.0, 4.0, 5.0])
    B = CSR.from_coo(4, 5, [0, 0, 3], [4, 1, 2], [10.0, 20.0, 30.0])
    got, _ = run_ttm(ctx, A, B, policy)
    assert list(got["crd0"]) == [0, 2] and list(got["pos1"]) == [0, 1, 2] and list(got["crd1"]) == [2, 1]
    assert list(got["pos2"]) == [0, 2, 3] and list(got["crd2"]) == [1, 4, 2] and list(got["val"]) == [40.0, 20.0, 150.0]
    for dims, nnz, seed in (((8, 8, 8), 100, 1), ((20, 30, 40), 3000, 2), ((64, 64, 64), 20000, 3)):
        A = uniform_csf3(dims, nnz, seed)
        B = random_csr(dims[2], 300, 0.05, seed + 5, empty_row_frac=0.5)
        check_ttm(ctx, oracle_mod, A, B, policy)
        check_ttm(ctx, oracle_mod, A, B, policy, **SMALL_ROUTES)


@pytest.mark.parametrize("policy", POLICIES)
@pytest.mark.parametrize("reduced", [True, False])
def test_ttm_config(ctx, oracle_mod, reduced, policy):
    c = config_inputs("ttm4096", reduced=reduced)
    stats = check_ttm(ctx, oracle_mod, c["A"], c["B"], policy)
    assert stats["products"] == 8 * c["A"].nnz


@pytest.mark.parametrize("slices", [4097, 9001, 70001])
def test_ttm_many_slices_and_dropped_fibres(ctx, oracle_mod, slices):
    """Slice levels of one and several 4096-slice rounds with a ragged tail, and beyond 2^16 slices
    (the multi-launch slice level); half of B's rows are empty, so many fibres and slices produce no
    output and drop out of C's upper levels; the fibre count spans several scan tiles."""
    A = uniform_csf3((slices, 50, 64), 3 * slices, 21)
    B = random_csr(64, 400, 0.05, 22, empty_row_frac=0.5)
    stats = check_ttm(ctx, oracle_mod, A, B, "auto")
    assert stats["rows"] > 2048


def test_ttm_equals_spgemm_of_the_fibre_matrix(ctx):
    """Hoisting the shared outer loops turns the 3-tensor form into the matrix form over the (i,j)
    fibres: the last CSF level of the TTM result must equal the CSR result of the fibre matrix times
    B on the same device path, bit for bit in structure and within rounding in value (fp32, fp64)."""
    for dtype in (np.float32, np.float64):
        A = uniform_csf3((48, 40, 64), 9000, 4)
        A.val = A.val.astype(dtype)
        B = random_csr(64, 500, 0.1, 9, empty_row_frac=0.3)
        B.val = B.val.astype(dtype)
        got, _ = run_ttm(ctx, A, B, "auto")
        pos, crd, val, _ = run_spgemm(ctx, A.fibres_as_csr(), B, "auto")
        keep = np.diff(pos) > 0                     # fibres without an output are dropped from C
        assert np.array_equal(got["pos2"], np.concatenate([[0], np.cumsum(np.diff(pos)[keep])]))
        assert np.array_equal(got["crd2"], crd)
        tol = TOL[np.dtype(dtype)]                  # routes with atomics sum in a run-dependent order
        assert np.allclose(got["val"], val, rtol=100 * tol, atol=100 * tol)
        assert np.array_equal(got["crd1"], A.crd1[keep])


def test_execute_host_ttm_and_distinct_operands(ctx, oracle_mod):
    """The host-buffer entry point on the 3-tensor form and on a matrix product with B != A."""
    import torch
    from paper_2404_04541_b200 import api, binding
    arena = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    A = uniform_csf3((32, 32, 64), 6000, 7)
    B = random_csr(64, 200, 0.1, 8, empty_row_frac=0.4)
    ref = oracle_mod.ttm(A, B)
    plan = ctx.plan(api.EXPR_TTM, (binding.SPWS_CSF3, binding.SPWS_CSF3, binding.SPWS_CSR), np.float64)
    a = binding.csf3_arrays(A.dims, A.pos0, A.crd0, A.pos1, A.crd1, A.pos2, A.crd2, A.val)
    b = binding.csr_arrays(B.nrows, B.ncols, B.pos, B.crd, B.val)
    nnz = ref.crd2.shape[0]
    out = dict(pos0=np.empty(2, np.int64), crd0=np.empty(A.n_i, np.int32), pos1=np.empty(A.n_i + 1, np.int64),
               crd1=np.empty(A.n_ij, np.int32), pos2=np.empty(A.n_ij + 1, np.int64), crd2=np.empty(nnz, np.int32),
               val=np.empty(nnz, np.float64))
    c = binding.TensorArrays(3, (A.dims[0], A.dims[1], B.ncols), [out["pos0"], out["pos1"], out["pos2"]],
                             [out["crd0"], out["crd1"], out["crd2"]], out["val"], [A.n_i, A.n_ij, nnz])
    st, sizes, _ = plan.execute_host(a, b, c, ctx._aligned_ptr(arena), arena.numel() - 256)
    assert st == 0 and sizes == [ref.crd0.shape[0], ref.crd1.shape[0], nnz]
    assert np.array_equal(out["pos0"], ref.pos0) and np.array_equal(out["crd0"][:sizes[0]], ref.crd0)
    assert np.array_equal(out["pos1"][:sizes[0] + 1], ref.pos1) and np.array_equal(out["crd1"][:sizes[1]], ref.crd1)
    assert np.array_equal(out["pos2"][:sizes[1] + 1], ref.pos2) and np.array_equal(out["crd2"], ref.crd2)
    ok, _ = values_close(out["val"], ref.val_ref, ref.abs, 1e-12)
    assert ok.all()
    plan.close()
    # matrix form, two different operands
    M, N = random_csr(300, 64, 0.1, 12), B
    mref = oracle_mod.spgemm(M, N)
    plan = ctx.plan(api.EXPR_SPGEMM, (0, 0, 0), np.float64)
    cpos, ccrd, cval = np.empty(301, np.int64), np.empty(mref.nnz, np.int32), np.empty(mref.nnz, np.float64)
    cm = binding.csr_arrays(300, N.ncols, cpos, ccrd, cval)
    st, sizes, _ = plan.execute_host(binding.csr_arrays(300, 64, M.pos, M.crd, M.val), b, cm, ctx._aligned_ptr(arena),
                                     arena.numel() - 256)
    assert st == 0 and sizes[1] == mref.nnz
    assert np.array_equal(cpos, mref.pos) and np.array_equal(ccrd, mref.crd)
    ok, _ = values_close(cval, mref.val_ref, mref.abs, 1e-12)
    assert ok.all()
    plan.close()


# ------------------------------------------------------------------ exact scratch sizing
@pytest.mark.parametrize("policy", ["auto", "dense", "ism"])
def test_exact_workspace_size_suffices_and_is_tight(ctx, oracle_mod, policy):
    """spws_workspace_size_exact returns what both passes use: the result is right with exactly
    that much scratch, a buffer 256 bytes shorter is refused, and the figure is far below the
    host-side upper bound when rows are narrower than the matrix."""
    import torch
    from paper_2404_04541_b200 import api, binding
    A = rmat_csr(12, 16, 9)
    dA = api.DeviceCSR.from_host(A)
    a = dA.arrays()
    plan = ctx.plan(api.EXPR_SPGEMM, (binding.SPWS_CSR,) * 3, np.float64, policy, ism_cta_cap=256, fallback_cap=64)
    upper = plan.workspace_size(a, a)
    own = plan.workspace_size_exact(a, a)
    assert 0 < own <= upper
    buf = torch.empty(upper + 256, dtype=torch.uint8, device="cuda")
    ptr = ctx._aligned_ptr(buf)
    ub_dev = torch.empty(A.nrows, dtype=torch.int64, device="cuda")
    exact = plan.workspace_size_exact(a, a, ptr, own, ub_dev.data_ptr())
    assert own <= exact <= upper
    lens = np.diff(A.pos)
    ub = np.bincount(rows_of(A.pos), weights=lens[A.crd], minlength=A.nrows).astype(np.int64)
    assert np.array_equal(ub_dev.cpu().numpy(), ub)
    if policy != "ism":
        assert exact < upper
    pos = torch.empty(A.nrows + 1, dtype=torch.int64, device="cuda")
    c = binding.csr_arrays(A.nrows, A.ncols, pos, None, None)
    plan.symbolic(a, a, c, ptr, exact)
    ref = oracle_mod.spgemm(A, A, threads=4)
    nnz = c.n[1]
    assert nnz == ref.nnz
    c.crd[1] = torch.empty(nnz, dtype=torch.int32, device="cuda")
    c.val = torch.empty(nnz, dtype=torch.float64, device="cuda")
    plan.numeric(a, a, c, ptr, exact)
    stats = plan.get_stats()                                         # reports a device-side failure, if any
    assert_matches((pos.cpu().numpy(), c.crd[1].cpu().numpy(), c.val.cpu().numpy()), ref, np.float64)
    if policy != "ism" and exact > own:                              # bitmaps in use: a shorter arena cannot hold them
        with pytest.raises(binding.SpwsError) as e:
            plan.symbolic(a, a, c, ptr, exact - 256)
            plan.numeric(a, a, c, ptr, exact - 256)
            plan.get_stats()
        assert e.value.status == binding.SPWS_SCRATCH_TOO_SMALL
    plan.close()


# ------------------------------------------------------------------ boundary behaviour
def test_error_statuses(ctx):
    import torch
    from paper_2404_04541_b200 import api, binding
    with pytest.raises(binding.SpwsError) as e:
        ctx.plan("C(i,j) = A(i,k) * B(j,k)", (0, 0, 0), np.float64)
    assert e.value.status == binding.SPWS_UNSUPPORTED_EXPRESSION
    A = api.DeviceCSR.from_host(random_csr(10, 12, 0.3, 1))
    Bm = api.DeviceCSR.from_host(random_csr(13, 9, 0.3, 2))
    with pytest.raises(binding.SpwsError) as e:
        ctx.spgemm(A, Bm)
    assert e.value.status == binding.SPWS_DIM_MISMATCH
    # scratch too small / numeric before symbolic
    plan = ctx.plan(api.EXPR_SPGEMM, (0, 0, 0), np.float64)
    Bok = api.DeviceCSR.from_host(random_csr(12, 9, 0.3, 2))
    a, b = A.arrays(), Bok.arrays()
    pos = torch.empty(11, dtype=torch.int64, device="cuda")
    c = binding.csr_arrays(10, 9, pos, None, None)
    sc = ctx.scratch(plan.workspace_size(a, b))
    with pytest.raises(binding.SpwsError) as e:
        plan.symbolic(a, b, c, ctx._aligned_ptr(sc), 64)
    assert e.value.status == binding.SPWS_SCRATCH_TOO_SMALL
    with pytest.raises(binding.SpwsError) as e:
        plan.numeric(a, b, c, ctx._aligned_ptr(sc), plan.workspace_size(a, b))
    assert e.value.status == binding.SPWS_BAD_SEQUENCE
    plan.close()
    # non-canonical input is reported when validation is on
    bad = random_csr(12, 9, 0.6, 3)
    bad.crd[0], bad.crd[1] = bad.crd[1], bad.crd[0]
    with pytest.raises(binding.SpwsError) as e:
        ctx.spgemm(A, api.DeviceCSR.from_host(bad), validate=1)
    assert e.value.status == binding.SPWS_NONCANONICAL_INPUT
    oob = random_csr(10, 12, 0.3, 1)
    oob.crd[2] = 12
    with pytest.raises(binding.SpwsError) as e:
        ctx.spgemm(api.DeviceCSR.from_host(oob), Bok)
    assert e.value.status == binding.SPWS_NONCANONICAL_INPUT


def test_execute_host_matches(ctx, oracle_mod):
    import torch
    from paper_2404_04541_b200 import api, binding
    A = rmat_csr(10, 8, 3)
    ref = oracle_mod.spgemm(A, A)
    plan = ctx.plan(api.EXPR_SPGEMM, (0, 0, 0), np.float64)
    a = binding.csr_arrays(A.nrows, A.ncols, A.pos, A.crd, A.val)
    cpos = np.empty(A.nrows + 1, dtype=np.int64)
    ccrd = np.empty(ref.nnz + 10, dtype=np.int32)
    cval = np.empty(ref.nnz + 10, dtype=np.float64)
    c = binding.csr_arrays(A.nrows, A.ncols, cpos, ccrd, cval)
    arena = torch.empty(256 << 20, dtype=torch.uint8, device="cuda")
    st, sizes, need = plan.execute_host(a, a, c, ctx._aligned_ptr(arena), arena.numel() - 256)
    assert st == 0 and sizes[1] == ref.nnz and 0 < need <= arena.numel()
    assert np.array_equal(cpos, ref.pos) and np.array_equal(ccrd[:ref.nnz], ref.crd)
    ok, _ = values_close(cval[:ref.nnz], ref.val_ref, ref.abs, 1e-12)
    assert ok.all()
    c.n = [A.nrows, 5, 0]                                              # capacity too small
    st, sizes, _ = plan.execute_host(a, a, c, ctx._aligned_ptr(arena), arena.numel() - 256)
    assert st == binding.SPWS_OUTPUT_TOO_SMALL and sizes[1] == ref.nnz
    plan.close()
