"""Row-sharded SpGEMM across ranks (host logic).

Output rows are independent (row-wise SpGEMM is a first-order scatter, Sec. 2.2: nothing crosses
rows), so A is cut into contiguous row blocks, B is replicated, every rank runs the unchanged
single-GPU path on its block, and the only exchange is an all-gather of each rank's output size
to place its row-pointer slice.  No collective touches the data path.

The local product and the per-row product counts the partition balances on are passed in as
callables, so that the same code drives the CUDA path (`local_spgemm_cuda`, `row_products_cuda`:
the counts come from the symbolic pass's first kernel on the device) and, in CPU tests, stand-ins.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable

import numpy as np
import torch
import torch.distributed as dist


def partition_rows(weights: np.ndarray, world: int) -> np.ndarray:
    """Boundaries r[0..world] of contiguous row blocks with nearly equal total weight (+1 per
    row so that empty rows are spread as well)."""
    w = weights.astype(np.float64) + 1.0
    csum = np.concatenate([[0.0], np.cumsum(w)])
    targets = csum[-1] * np.arange(1, world) / world
    cuts = np.searchsorted(csum, targets, side="left")
    bounds = np.concatenate([[0], cuts, [weights.shape[0]]]).astype(np.int64)
    return np.maximum.accumulate(bounds)


@dataclass
class ShardResult:
    row_begin: int
    row_end: int
    pos: np.ndarray       # GLOBAL row pointer values of this rank's rows: pos[0] = entries before this rank
    crd: np.ndarray
    val: np.ndarray
    nnz_per_rank: np.ndarray


def spgemm_sharded(A, B, local_spgemm: Callable, row_products: Callable, group=None) -> ShardResult:
    """Each rank multiplies its row block of A by the replicated B.

    `A`, `B` are host CSR containers (attributes nrows, ncols, pos, crd, val and row_block);
    `local_spgemm(A_block, B)` returns (pos, crd, val) numpy arrays of the block's product;
    `row_products(A, B)` returns the int64 product count of every row of A (every rank computes
    the same partition from it).
    """
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    bounds = partition_rows(np.asarray(row_products(A, B), dtype=np.int64), world)
    r0, r1 = int(bounds[rank]), int(bounds[rank + 1])
    pos, crd, val = local_spgemm(A.row_block(r0, r1), B)
    mine = torch.tensor([int(pos[-1])], dtype=torch.int64)
    everyone = [torch.zeros(1, dtype=torch.int64) for _ in range(world)]
    dist.all_gather(everyone, mine, group=group)
    nnz = np.array([int(t.item()) for t in everyone], dtype=np.int64)
    before = int(nnz[:rank].sum())
    return ShardResult(r0, r1, np.asarray(pos, dtype=np.int64) + before, crd, val, nnz)


def gather_full(res: ShardResult, nrows: int, group=None):
    """Concatenate every rank's block on all ranks (for checks and small outputs)."""
    world = dist.get_world_size(group)
    parts = [None] * world
    dist.all_gather_object(parts, (res.row_begin, res.row_end, res.pos, res.crd, res.val), group=group)
    parts.sort(key=lambda p: p[0])
    pos = np.zeros(nrows + 1, dtype=np.int64)
    for r0, r1, p, _, _ in parts:
        pos[r0:r1 + 1] = p
    crd = np.concatenate([p[3] for p in parts]) if parts else np.zeros(0, np.int32)
    val = np.concatenate([p[4] for p in parts]) if parts else np.zeros(0)
    return pos, crd, val


def local_spgemm_cuda(ctx, policy: str = "auto", **options) -> Callable:
    """The CUDA path as the local product: uploads the block, runs symbolic + numeric."""
    from . import api

    def run(A_block, B):
        dA = api.DeviceCSR.from_host(A_block, device=ctx.device)
        dB = api.DeviceCSR.from_host(B, device=ctx.device)
        C, _ = ctx.spgemm(dA, dB, policy=policy, **options)
        return C.pos.cpu().numpy(), C.crd.cpu().numpy(), C.val.cpu().numpy()

    return run


def row_products_cuda(ctx) -> Callable:
    """Per-row product counts from the device: the upper-bound kernel of the symbolic pass, run by
    the exact-sizing entry point."""
    from . import api
    from . import binding as B_

    def run(A, B):
        dA = api.DeviceCSR.from_host(A, device=ctx.device)
        dB = api.DeviceCSR.from_host(B, device=ctx.device)
        dt = np.float64 if dA.val.dtype == torch.float64 else np.float32
        plan = ctx.plan(api.EXPR_SPGEMM, (B_.SPWS_CSR,) * 3, dt, "auto")
        try:
            ub = torch.empty(max(A.nrows, 1), dtype=torch.int64, device=ctx.device)
            ctx.exact_scratch_bytes(plan, dA.arrays(), dB.arrays(), row_products=ub)
            return ub[:A.nrows].cpu().numpy()
        finally:
            plan.close()

    return run
