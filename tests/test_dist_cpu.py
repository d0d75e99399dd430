"""Row-sharded driver on CPU: two gloo ranks, the local product supplied by the oracle (the
host logic under test is the partition, the size exchange and the row-pointer offsets)."""
import os
import socket
import sys

import numpy as np
import pytest
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _worker(rank, world, port, out_dir):
    sys.path.insert(0, ROOT)
    import torch.distributed as dist
    import oracle
    from paper_2404_04541_b200 import dist as spd
    from workloads import rmat_csr
    dist.init_process_group("gloo", init_method=f"tcp://127.0.0.1:{port}", rank=rank, world_size=world)
    A = rmat_csr(9, 8, 4)

    def local(Ab, B):
        r = oracle.spgemm(Ab, B)
        return r.pos, r.crd, r.val

    def products(Am, Bm):                       # stand-in for the device's per-row product counts
        return oracle.spgemm(Am, Bm).products

    res = spd.spgemm_sharded(A, A, local, products)
    pos, crd, val = spd.gather_full(res, A.nrows)
    np.savez(os.path.join(out_dir, f"rank{rank}.npz"), pos=pos, crd=crd, val=val, r0=res.row_begin, r1=res.row_end,
             nnz=res.nnz_per_rank, first=res.pos[0])
    dist.destroy_process_group()


def test_partition_balances_weights():
    from paper_2404_04541_b200.dist import partition_rows
    w = np.array([0, 0, 100, 1, 1, 1, 100, 0, 0, 0], dtype=np.int64)
    b = partition_rows(w, 2)
    assert b[0] == 0 and b[-1] == 10 and (np.diff(b) >= 0).all()
    left, right = w[:b[1]].sum(), w[b[1]:].sum()
    assert abs(left - right) <= 100
    assert list(partition_rows(np.zeros(5, dtype=np.int64), 5)) == [0, 1, 2, 3, 4, 5]
    assert partition_rows(np.ones(3, dtype=np.int64), 8)[-1] == 3       # more ranks than rows: empty blocks


def test_two_rank_sharded_spgemm_matches_unsharded(tmp_path, oracle_mod):
    from workloads import rmat_csr
    port = _free_port()
    mp.spawn(_worker, args=(2, port, str(tmp_path)), nprocs=2, join=True)
    A = rmat_csr(9, 8, 4)
    ref = oracle_mod.spgemm(A, A)
    outs = [np.load(os.path.join(str(tmp_path), f"rank{r}.npz")) for r in range(2)]
    for o in outs:
        assert np.array_equal(o["pos"], ref.pos) and np.array_equal(o["crd"], ref.crd) and np.array_equal(o["val"], ref.val)
    assert outs[0]["r0"] == 0 and outs[0]["r1"] == outs[1]["r0"] and outs[1]["r1"] == A.nrows
    assert outs[0]["first"] == 0 and outs[1]["first"] == outs[0]["nnz"][0]
    assert outs[0]["nnz"].sum() == ref.nnz
