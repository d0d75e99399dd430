"""Shared helpers for the tests: golden-file parsing, comparison rules."""
from __future__ import annotations

import os

import numpy as np

from workloads import CSR

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")

# Tolerances of the parity bar: relative error per entry.  A sum of mixed-sign products can
# cancel, so an entry also passes when the error is within tol * sum|a*b| (the forward error
# scale of a reordered summation).
TOL = {np.dtype(np.float64): 1e-12, np.dtype(np.float32): 1e-5}


def read_hand_case(name: str):
    """Parse a hand-worked case: returns (A, B, C_rows, C_cols, C_vals, products)."""
    ent = {"A": [], "B": [], "C": []}
    shape = products = None
    with open(os.path.join(GOLDEN, name)) as f:
        for line in f:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            tok = line.split()
            if tok[0] == "shape":
                shape = tuple(int(t) for t in tok[1:])
            elif tok[0] == "products":
                products = np.array([int(t) for t in tok[1:]], dtype=np.int64)
            else:
                ent[tok[0]].append((int(tok[1]), int(tok[2]), float(tok[3])))
    m, k, n = shape

    def mk(rows, cols, es):
        r = [e[0] for e in es]
        c = [e[1] for e in es]
        v = [e[2] for e in es]
        return CSR.from_coo(rows, cols, r, c, v)

    C = sorted(ent["C"])
    return (mk(m, k, ent["A"]), mk(k, n, ent["B"]),
            np.array([e[0] for e in C]), np.array([e[1] for e in C]),
            np.array([e[2] for e in C], dtype=np.float64), products)


def rows_of(pos: np.ndarray) -> np.ndarray:
    return np.repeat(np.arange(pos.shape[0] - 1), np.diff(pos))


def values_close(got: np.ndarray, ref: np.ndarray, absum: np.ndarray, tol: float):
    """Per-entry pass mask under the two-clause rule; returns (ok_mask, n_needing_second_clause)."""
    got = got.astype(np.float64)
    err = np.abs(got - ref)
    first = err <= tol * np.abs(ref)
    second = err <= tol * absum
    return first | second, int((~first & second).sum())
