"""Seeded synthetic inputs (CSR matrices, CSF 3-tensors) shaped like the paper's workloads.

This module is shared test/bench harness: it builds operands only.  It holds none of the
method's arithmetic (no products, no accumulation, no workspaces) and imports neither the
oracle nor the CUDA binding.
"""
from .formats import CSR, CSF3, csr_is_canonical, csf3_is_canonical
from .generators import (
    uniform_rows_csr,
    rmat_csr,
    stencil27_csr,
    uniform_csf3,
    random_csr,
    crossover_operands,
    config_inputs,
    CONFIG_NAMES,
)

__all__ = [
    "CSR", "CSF3", "csr_is_canonical", "csf3_is_canonical",
    "uniform_rows_csr", "rmat_csr", "stencil27_csr", "uniform_csf3", "random_csr", "crossover_operands",
    "config_inputs", "CONFIG_NAMES",
]
