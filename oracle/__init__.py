"""CPU oracle (test infrastructure only): see oracle.cpp for what each entry computes.

Only the tests, the smoke check and the benchmark's CPU-baseline / reference legs may import
this package.  It does not import the CUDA binding and the binding does not import it.
"""
from .oracle import (build, spgemm, ttm, ism_rowwise, ism_outer, hardware_threads,
                     SpgemmResult, TtmResult)
from .higher import spttm, spttm_i, spmttkrp, CooResult

__all__ = ["build", "spgemm", "ttm", "ism_rowwise", "ism_outer", "hardware_threads",
           "SpgemmResult", "TtmResult", "spttm", "spttm_i", "spmttkrp", "CooResult"]
