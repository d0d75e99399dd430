"""spws: sparse-workspace SpGEMM / TTM kernels for NVIDIA B200 behind a C ABI (include/spws.h).

`binding` mirrors the C entry points (ctypes); `api` adds torch-allocated convenience calls;
`build` compiles the library in-tree.  The package has no CPU path.
"""
from . import binding  # noqa: F401

__all__ = ["binding"]
