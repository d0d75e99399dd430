"""Row-sharded SpGEMM across ranks (host logic).

Output rows are independent (row-wise SpGEMM is a first-order scatter, Sec. 2.2: nothing crosses
rows), so A is cut into contiguous row blocks, B is replicated, every rank runs the unchanged
single-GPU path on its block, and the only exchange is an all-gather of each rank's output size
to place its row-pointer slice.  No collective touches the data path.

The local product is passed in as a callable so that the same code drives the CUDA path
(`local_spgemm_cuda`) and, in CPU tests, a stand-in.
"""
from __future__ import annotations

from dataclasses import dataclass
from typing import Callable

import numpy as np
import torch
import torch.distributed as dist


def row_weights(A_pos: np.ndarray, A_crd: np.ndarray, B_pos: np.ndarray) -> np.ndarray:
    """Per-row product upper bound (the symbolic pass's first quantity), on the host."""
    blen = np.diff(B_pos)
    rows = np.repeat(np.arange(A_pos.shape[0] - 1), np.diff(A_pos))
    return np.bincount(rows, weights=blen[A_crd], minlength=A_pos.shape[0] - 1).astype(np.int64)


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


def spgemm_sharded(A, B, local_spgemm: Callable, group=None) -> ShardResult:
    """Each rank multiplies its row block of A by the replicated B.

    `A`, `B` are host CSR containers (attributes nrows, ncols, pos, crd, val and row_block);
    `local_spgemm(A_block, B)` returns (pos, crd, val) numpy arrays of the block's product.
    """
    world = dist.get_world_size(group)
    rank = dist.get_rank(group)
    bounds = partition_rows(row_weights(A.pos, A.crd, B.pos), world)
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
