#!/usr/bin/env python
"""Benchmark of the sparse-workspace SpGEMM path on B200.

One step = one whole pass of the hot path (symbolic + numeric, policy auto) over one synthetic
operand set already resident in HBM.  Default workload: the power-law configuration (R-MAT,
2^18 vertices, average degree 16, C = A*A, fp64).  Prints ONE JSON line on rank 0.

    python bench.py [--gpus N] [--steps K] [--warmup W] [--workload NAME] [--impl reference]

N > 1 (under torchrun): ONE seeded problem; every rank takes a contiguous block of A's rows,
balanced on the per-row product counts the device computes, with B replicated (output rows are
independent, so the only exchange is an all-gather of the ranks' output sizes); value = the
whole problem's flops over the slowest rank's device time ("scaling": "strong").
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import tempfile
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC, UNIT = "spgemm_gflops_2_per_product", "GFLOP/s"
WORKLOAD_TEXT = {
    "rmat18": "power-law SpGEMM C=A*A, R-MAT 2^18 vertices, degree 16, (0.57,0.19,0.19,0.05), fp64",
    "stencil64": "FEM-like SpGEMM C=A*A, 27-point stencil on 64^3, fp64",
    "uniform8": "SpGEMM C=A*A, 2048x2048, 8 nnz/row, fp64",
    "wide26": "wide-output SpGEMM, A 65536 x 2^26, B 2^26 x 2^26, 4 nnz/row, fp32",
    "ttm4096": "3-tensor times matrix C(i,j,l)=A(i,j,k)B(k,l), A 4096^3 CSF with 2^21 nnz, B 4096^2 CSR 8 nnz/row, fp64",
}
NOMINAL_HBM_GBS = 8000.0
# DRAM traffic (dram__bytes_read.sum + dram__bytes_write.sum) per product of the two kernels that
# dominate the default and the stencil workloads, from the ncu captures summarised under
# profiles/ (taken on a smaller case of the same recipe where noted; traffic grows in proportion
# to the products).  Valid only for the kernel source the capture was taken on.
PROFILED_TRAFFIC = {
    "num_dense_cta": {"bytes_per_product": (2399641000 + 3737405000) / 1085650666, "source": "profiles/dense_cta_kernels_rmat17.md"},
    "num_dense_warp": {"bytes_per_product": (328682752 + 332724736) / 181321496, "source": "profiles/dense_warp_kernels_stencil64.md"},
}
PROFILED_SOURCE_SHA = "f7c7ee0c3c373669"   # sha256 prefix of csrc/dense.cu at capture time


def algorithmic_bytes(m, nnzA, products, nnzC, V):
    """Bytes the method itself must move, counted once: A read, gathered B rows (two offsets per
    A entry + index and value per product), C written."""
    return ((m + 1) * 8 + nnzA * (4 + V)) + (nnzA * 16 + products * (4 + V)) + ((m + 1) * 8 + nnzC * (4 + V))


def measured_peak():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""
    QUERY = ("index,clocks.sm,clocks.max.sm,power.draw,clocks_event_reasons.active,"
             "clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
             "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, gpu_index: int):
        self.gpu = gpu_index
        self.proc = None
        self.path = None

    def start(self):
        try:
            fd, self.path = tempfile.mkstemp(suffix=".csv")
            os.close(fd)
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.QUERY}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.gpu)],
                                         stdout=open(self.path, "w"), stderr=subprocess.DEVNULL)
        except Exception:
            self.proc = None

    def stop(self) -> dict:
        out = {"sm_mhz": None, "sm_max_mhz": None, "reasons": [], "samples": 0}
        if self.proc is None:
            return out
        time.sleep(0.15)
        self.proc.terminate()
        try:
            self.proc.wait(timeout=5)
        except Exception:
            self.proc.kill()
        sm, mx, reasons = [], [], set()
        try:
            for line in open(self.path):
                f = [x.strip() for x in line.split(",")]
                if len(f) < 9:
                    continue
                try:
                    sm.append(float(f[1])); mx.append(float(f[2]))
                except ValueError:
                    continue
                for name, v in zip(("hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"), f[5:9]):
                    if v.lower().startswith("active"):
                        reasons.add(name)
            os.unlink(self.path)
        except Exception:
            pass
        if sm:
            out.update(sm_mhz=float(np.median(sm)), sm_max_mhz=float(max(mx)), reasons=sorted(reasons), samples=len(sm))
        return out


def oracle_sample(A, B, budget_products: float, seed: int = 0):
    """Rows of the workload drawn at random until their products reach the budget."""
    rng = np.random.default_rng(seed)
    lens = np.diff(B.pos)
    rows_of_nz = np.repeat(np.arange(A.nrows), np.diff(A.pos))
    ub = np.bincount(rows_of_nz, weights=lens[A.crd], minlength=A.nrows).astype(np.int64)
    order = rng.permutation(A.nrows)
    csum = np.cumsum(ub[order])
    n = int(np.searchsorted(csum, budget_products) + 1)
    n = max(1, min(n, A.nrows))
    rows = np.sort(order[:n])
    return rows, int(ub[rows].sum()), int(ub.sum())


def time_oracle(A, B, rows, threads):
    import oracle
    t0 = time.perf_counter()
    res = oracle.spgemm(A, B, rows=rows, threads=threads)
    dt = time.perf_counter() - t0
    return dt, int(res.products.sum())


def sized_oracle_sample(A, B, threads, seconds):
    """Calibrate on a small sample, then size a sample for about `seconds` of CPU work."""
    rows0, p0, total = oracle_sample(A, B, 2e7)
    dt0, _ = time_oracle(A, B, rows0, threads)
    budget = min(total, max(2e7, p0 / max(dt0, 1e-6) * seconds))
    rows, psample, _ = oracle_sample(A, B, budget)
    return rows, psample, total


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on the host cores, on a bounded sample."""
    if int(os.environ.get("RANK", "0")) != 0:
        return
    import oracle
    from workloads import config_inputs
    oracle.build()
    cfg = config_inputs(args.workload, seed=args.seed)
    A, B = cfg["A"], cfg["B"]
    if cfg["kind"] == "ttm":                     # the 3-tensor form is the matrix form over the (i,j) fibres
        A = A.fibres_as_csr()
    threads = oracle.hardware_threads()
    rows, psample, total = sized_oracle_sample(A, B, threads, 6.0)
    for _ in range(args.warmup):
        time_oracle(A, B, rows, threads)
    times = [time_oracle(A, B, rows, threads)[0] for _ in range(args.steps)]
    ms = 1e3 * float(np.mean(times))
    value = 2.0 * psample / (ms * 1e-3) / 1e9
    sample = f"{rows.size} random rows of {A.nrows}, {psample} of {total} products per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "f64", "data": "synthetic",
            "config": {"workload": WORKLOAD_TEXT[args.workload], "name": args.workload, "seed": args.seed,
                       "sample": sample},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": threads, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)


def percentile_stats(xs):
    xs = sorted(xs)
    return float(np.mean(xs)), float(xs[0]), float(np.median(xs))


def measure(workload, args, dev, rank, world, dist, e2e=True, cpu_baseline=True):
    """Times `args.steps` steps of symbolic + numeric on one workload; returns the fields of the
    bench line that belong to the workload."""
    import torch
    from paper_2404_04541_b200 import api, binding
    from workloads import config_inputs

    WORKLOAD_TEXT.setdefault(workload, f"{workload} (same recipe as the named configuration, other size), fp64")
    is_ttm = workload.startswith("ttm")
    # N > 1, matrix form: ONE seeded problem; every rank takes a block of A's rows, balanced on the
    # per-row product counts, with B replicated (output rows are independent).  The 3-tensor form
    # keeps one problem per rank.
    sharded = world > 1 and not is_ttm
    cfg = config_inputs(workload, seed=args.seed + (0 if sharded else rank))
    T3 = cfg["A"] if is_ttm else None           # the CSF operand of the 3-tensor form
    # the 3-tensor form works on the (i,j) fibres as rows: sizes, bytes and the oracle sample use that matrix
    A, B = (T3.fibres_as_csr() if is_ttm else cfg["A"]), cfg["B"]
    V = 8 if cfg["dtype"] == np.float64 else 4
    vt = torch.float64 if V == 8 else torch.float32
    ctx = api.Context(dev)
    row_block = None
    if sharded:
        from paper_2404_04541_b200 import dist as spd
        bounds = spd.partition_rows(spd.row_products_cuda(ctx)(A, B), world)
        row_block = (int(bounds[rank]), int(bounds[rank + 1]))
        A = A.row_block(*row_block)
    options = {}
    for kv in args.opt:
        name, value = kv.split("=", 1)
        options[name] = float(value) if "." in value else int(value)
    if is_ttm:
        dA = api.DeviceCSF3.from_host(T3, dev)
        dB = api.DeviceCSR.from_host(B, device=dev)
        plan = ctx.plan(api.EXPR_TTM, (binding.SPWS_CSF3, binding.SPWS_CSF3, binding.SPWS_CSR), cfg["dtype"], args.policy, **options)
        symbolic, numeric, last = ctx.ttm_symbolic, ctx.ttm_numeric, 2
    else:
        dA = api.DeviceCSR.from_host(A, device=dev)
        dB = dA if B is A else api.DeviceCSR.from_host(B, device=dev)
        plan = ctx.plan(api.EXPR_SPGEMM, (binding.SPWS_CSR,) * 3, cfg["dtype"], args.policy, **options)
        symbolic, numeric, last = ctx.spgemm_symbolic, ctx.spgemm_numeric, 1
    plan.set_profiling(True)

    # a first pass sizes C; its buffers are reused by every step (allocation is outside the timed region)
    c, state = symbolic(plan, dA, dB)
    nnzC = c.n[last]
    crd = torch.empty(nnzC, dtype=torch.int32, device=dev)
    val = torch.empty(nnzC, dtype=vt, device=dev)
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)       # > L2 (126 MB)
    result = {}

    nnz_all = torch.zeros(world, dtype=torch.int64, device=dev)

    def step():
        cc, st = symbolic(plan, dA, dB)
        result["C"] = numeric(plan, cc, st, crd=crd, val=val)
        result["c"], result["state"] = cc, st
        if sharded:                                  # the one exchange: every rank's output size, to place its row pointers
            dist.all_gather_into_tensor(nnz_all, torch.tensor([cc.n[last]], dtype=torch.int64, device=dev))

    for _ in range(args.warmup):
        step()
    torch.cuda.synchronize()
    stats = plan.get_stats()
    products = stats["products"]

    sampler = ClockSampler(dev.index or 0)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(args.steps)]
    group_ms = {g: 0.0 for g in binding.TIMING_GROUPS}
    for s in range(args.steps):
        flush.fill_(s & 0xff)                                            # L2 flush between timed steps
        ev[s][0].record()
        step()
        ev[s][1].record()
        for g, ms in plan.get_timings().items():                         # synchronises the stream
            if not g.startswith("ceil_"):
                group_ms[g] += ms
    torch.cuda.synchronize()
    if world > 1:
        dist.barrier()
    clocks = sampler.stop()
    step_ms = [a.elapsed_time(b) for a, b in ev]
    total_ms = sum(step_ms)
    t = torch.tensor([total_ms, float(products), float(nnzC), float(A.nnz), float(A.nrows)], dtype=torch.float64, device=dev)
    if world > 1:
        tmax = t.clone()
        dist.all_reduce(tmax, op=dist.ReduceOp.MAX)
        dist.all_reduce(t, op=dist.ReduceOp.SUM)
        total_ms = float(tmax[0])
    all_products, all_nnzC, all_nnzA, all_m = float(t[1]), float(t[2]), float(t[3]), float(t[4])
    ms_per_step = total_ms / args.steps
    _, ms_min, ms_median = percentile_stats(step_ms)
    value = 2.0 * all_products / (ms_per_step * 1e-3) / 1e9
    abytes = algorithmic_bytes(all_m, all_nnzA, all_products, all_nnzC, V)
    eff_gbs = abytes / (ms_per_step * 1e-3) / 1e9

    # ---- iteration-only ceiling of the dense numeric kernels (outside the timed steps): the same
    # traversal and gathers with the workspace stripped
    ceil_ms = {"ceil_dense_warp": 0.0, "ceil_dense_cta": 0.0}
    if stats["dense_units"] > 0 or stats["dense_warp_rows"] > 0:
        n_ceil = max(1, min(args.steps, 5))
        for s in range(1 + n_ceil):
            flush.fill_(s & 0xff)
            ctx.gather_ceiling(plan, result["c"], result["state"])
            if s > 0:                                                    # first run is a warm-up
                tm = plan.get_timings()
                for g in ceil_ms:
                    ceil_ms[g] += tm[g] / n_ceil

    # ---- roofline of the dominant kernel (this rank's launches)
    peak, peak_kind = measured_peak()
    avg = {g: v / args.steps for g, v in group_ms.items() if not g.startswith("ceil_")}
    top = max(avg, key=avg.get)
    # algorithmic bytes of each per-class kernel group: numeric = index + value per product
    # gathered and per output written; symbolic = index per product gathered
    pc, nc = stats["products_per_class"], stats["nnz_per_class"]
    dw_p, dw_n = stats["dense_warp_products"], stats["dense_warp_nnz"]
    dense_p, dense_n = sum(pc[4:7]), sum(nc[4:7])
    group_units = {"ism_reg": (pc[1], nc[1]), "ism_smem_s": (pc[2], nc[2]), "ism_smem": (pc[3], nc[3]),
                   "ism_global": (pc[7], nc[7])}
    kname = top.split("_", 1)[1]
    if top == "num_dense_warp":
        kbytes = dw_p * (4 + V) + dw_n * (4 + V)
    elif top == "num_dense_cta":                    # gathers index + value per product, writes the values
        kbytes = (dense_p - dw_p) * (4 + V) + (dense_n - dw_n) * V
    elif top == "num_dense_emit":                   # writes the coordinates
        kbytes = (dense_n - dw_n) * 4
    elif top == "sym_dense_warp":
        kbytes = pc[4] * 4
    elif top == "sym_dense_cta":
        kbytes = (pc[5] + pc[6]) * 4
    else:
        gp, gn = group_units.get(kname, (0, 0))
        kbytes = gp * (4 + V) + gn * (4 + V) if top.startswith("num_") else gp * 4
    kunits = {"num_dense_cta": dense_p - dw_p, "num_dense_warp": dw_p}.get(top, 0)
    traffic = None
    if top in PROFILED_TRAFFIC and kunits:
        import hashlib
        src = os.path.join(ROOT, "paper_2404_04541_b200", "csrc", "dense.cu")
        if hashlib.sha256(open(src, "rb").read()).hexdigest().startswith(PROFILED_SOURCE_SHA):
            traffic = PROFILED_TRAFFIC[top]["bytes_per_product"] * kunits
    achieved = kbytes / (avg[top] * 1e-3) / 1e9 if avg[top] > 0 else 0.0
    ceiling = ceil_ms.get("ceil_" + top[len("num_"):]) if top.startswith("num_") else None
    roofline = {"bound": "hbm", "kernel": top, "achieved": achieved, "peak": peak, "unit": "GB/s",
                "frac": achieved / peak, "peak_kind": f"of {peak_kind}", "traffic": traffic,
                "kernel_ms": avg[top], "algorithmic_bytes": kbytes,
                # what the counters say limits this kernel: B is L2-resident, DRAM sees C and the saved bitmaps only
                "limiter": "SM load/store path (shared-memory atomics, L2 reductions, gather sectors), not DRAM",
                "dram_frac": (traffic / (avg[top] * 1e-3) / 1e9 / peak) if traffic else None,
                "ceiling_ms": ceiling, "kernel_over_ceiling": (avg[top] / ceiling) if ceiling else None,
                "ceiling": "same traversal and gathers, workspace stripped (spws_gather_ceiling)"}

    out = {"value": value, "ms_per_step": ms_per_step, "ms_min": ms_min, "ms_median": ms_median,
           "scaling": "strong" if sharded else "weak",
           "dtype": "f64" if V == 8 else "f32",
           "config": {"workload": WORKLOAD_TEXT[workload], "name": workload, "policy": args.policy, "options": options,
                      "seed": args.seed, "rows": int(A.nrows), "nnzA": int(A.nnz), "products": int(products),
                      "nnzC": int(nnzC), "l2": "512 MiB buffer written between timed steps",
                      "timed": "spws_symbolic + spws_numeric; C buffers preallocated" + ("; all-gather of the ranks' output sizes" if sharded else ""),
                      **({"sharding": f"rows {row_block[0]}..{row_block[1]} of one problem on rank {rank}; B replicated"} if sharded else {}),
                      **({"rows_are": "the (i,j) fibres of A"} if is_ttm else {})},
           "effective_gbs": eff_gbs, "algorithmic_bytes_per_step": abytes,
           "hbm_frac_nominal_8tbs": eff_gbs / NOMINAL_HBM_GBS, "hbm_frac_measured": eff_gbs / peak,
           "roofline": roofline, "kernel_ms": avg, "ceiling_ms": ceil_ms, "rows_per_class": stats["rows_per_class"],
           "products_per_class": stats["products_per_class"], "nnz_per_class": stats["nnz_per_class"],
           "dense_units": stats["dense_units"], "dense_warp_rows": stats["dense_warp_rows"],
           "bitmap_bytes": stats["bitmap_bytes"],
           "gpu_launches": (stats["launches_symbolic"] + stats["launches_numeric"]) * args.steps,
           "clocks": clocks}

    # ---- end to end through the host-buffer entry point (H2D of the operands, D2H of C inside the timed region)
    if e2e:
        try:
            keep = []

            def pin(a):
                t = torch.from_numpy(np.ascontiguousarray(a)).pin_memory()
                keep.append(t)
                return t.numpy()

            def pinned_out(n, dtype):
                t = torch.empty(max(int(n), 1), dtype=dtype).pin_memory()
                keep.append(t)
                return t.numpy()

            def host_csr(M):
                return binding.csr_arrays(M.nrows, M.ncols, pin(M.pos), pin(M.crd), pin(M.val))

            hb = host_csr(B)
            if is_ttm:
                ha = binding.csf3_arrays(T3.dims, pin(T3.pos0), pin(T3.crd0), pin(T3.pos1), pin(T3.crd1), pin(T3.pos2),
                                         pin(T3.crd2), pin(T3.val))
                n_i, n_ij = T3.n_i, T3.n_ij
                cc = binding.TensorArrays(3, (T3.dims[0], T3.dims[1], B.ncols),
                                          [pinned_out(2, torch.int64), pinned_out(n_i + 1, torch.int64), pinned_out(n_ij + 1, torch.int64)],
                                          [pinned_out(n_i, torch.int32), pinned_out(n_ij, torch.int32), pinned_out(nnzC, torch.int32)],
                                          pinned_out(nnzC, vt), [n_i, n_ij, nnzC])
                in_bytes = (16 + n_i * 4 + (n_i + 1) * 8 + n_ij * 4 + (n_ij + 1) * 8 + T3.nnz * (4 + V)
                            + (B.nrows + 1) * 8 + B.nnz * (4 + V))
                out_fixed = 16 + n_i * 4 + (n_i + 1) * 8 + n_ij * 4 + (n_ij + 1) * 8
            else:
                ha = hb if B is A else host_csr(A)
                cc = binding.csr_arrays(A.nrows, B.ncols, pinned_out(A.nrows + 1, torch.int64), pinned_out(nnzC, torch.int32),
                                        pinned_out(nnzC, vt))
                cc.n = [A.nrows, nnzC, 0]
                in_bytes = (A.nrows + 1) * 8 + A.nnz * (4 + V) + (0 if B is A else (B.nrows + 1) * 8 + B.nnz * (4 + V))
                out_fixed = (A.nrows + 1) * 8
            ws = plan.workspace_size(dA.arrays(), dB.arrays())
            arena_bytes = in_bytes + 2 * out_fixed + ws + nnzC * (4 + V) + (1 << 20)
            arena = torch.empty(arena_bytes + 256, dtype=torch.uint8, device=dev)
            aptr = ctx._aligned_ptr(arena)
            plan.set_profiling(False)
            for _ in range(2):
                st, sizes, need = plan.execute_host(ha, hb, cc, aptr, arena_bytes)
                if st != 0:
                    raise RuntimeError(f"execute_host: {binding.status_string(st)} (needs {need} bytes)")
            n_e2e = max(1, min(args.steps, 3))
            torch.cuda.synchronize()
            if world > 1:
                dist.barrier()
            e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
            e0.record()
            for _ in range(n_e2e):
                st, sizes, need = plan.execute_host(ha, hb, cc, aptr, arena_bytes)
            e1.record()
            torch.cuda.synchronize()
            e2e_ms = torch.tensor([e0.elapsed_time(e1) / n_e2e], dtype=torch.float64, device=dev)
            if world > 1:
                dist.all_reduce(e2e_ms, op=dist.ReduceOp.MAX)
            out_bytes = out_fixed + nnzC * (4 + V)
            out["e2e"] = {"value": 2.0 * all_products / (float(e2e_ms[0]) * 1e-3) / 1e9, "unit": UNIT,
                          "h2d_bytes_per_step": int(in_bytes), "d2h_bytes_per_step": int(out_bytes),
                          "ms_per_step": float(e2e_ms[0]), "steps": n_e2e,
                          "call": "spws_execute_host, pinned host buffers"}
            del arena
        except Exception as exc:  # report, do not hide
            out["e2e"] = {"value": None, "unit": UNIT, "error": str(exc)[:200]}

    # ---- the oracle timed on this machine's host cores, on a bounded sample (rank 0, N = 1); the same
    # sampled rows of the device result are compared with it entry by entry
    if cpu_baseline and rank == 0 and world == 1:
        import oracle
        oracle.build()
        threads = oracle.hardware_threads()
        rows, psample, total = sized_oracle_sample(A, B, threads, args.cpu_seconds)
        t0 = time.perf_counter()
        ref = oracle.spgemm(A, B, rows=rows, threads=threads)
        dt = time.perf_counter() - t0
        rows1, psample1, _ = oracle_sample(A, B, max(2e6, psample / max(dt, 1e-6) / max(threads, 1) * 3.0), seed=1)
        dt1, _ = time_oracle(A, B, rows1, 1)
        out["cpu_baseline"] = {"value": 2.0 * psample / dt / 1e9, "unit": UNIT, "cores": threads, "kind": "oracle",
                               "sample": f"{rows.size} random rows of {A.nrows}, {psample} of {total} products, {dt:.1f} s",
                               "single_thread": {"value": 2.0 * psample1 / dt1 / 1e9, "unit": UNIT, "cores": 1,
                                                 "sample": f"{rows1.size} random rows, {psample1} products, {dt1:.1f} s"}}
        # parity of the timed result on the sampled rows (structure exact; values under the two-clause rule)
        C = result["C"]
        pos = (C.pos2 if is_ttm else C.pos).cpu().numpy()
        dcrd, dval = (C.crd2, C.val) if is_ttm else (C.crd, C.val)
        tol = 1e-12 if V == 8 else 1e-5
        entries = second = bad = 0
        for tix, r in enumerate(rows):
            s0, s1 = int(pos[r]), int(pos[r + 1])
            u = slice(int(ref.pos[tix]), int(ref.pos[tix + 1]))
            got_c = dcrd[s0:s1].cpu().numpy()
            if got_c.shape[0] != u.stop - u.start or not np.array_equal(got_c, ref.crd[u]):
                bad += 1
                continue
            err = np.abs(dval[s0:s1].cpu().numpy().astype(np.float64) - ref.val_ref[u])
            first = err <= tol * np.abs(ref.val_ref[u])
            sec = err <= tol * ref.abs[u]
            bad += int((~(first | sec)).sum())
            second += int((~first & sec).sum())
            entries += u.stop - u.start
        out["parity_sample"] = {"rows": int(rows.size), "entries": int(entries), "mismatches": int(bad),
                                "second_clause_entries": int(second), "tolerance": tol}
    plan.close()
    return out


SWEEPS = {
    # Sec. 7.2, first-order workspaces: row-wise SpGEMM C = A*B, A is I x K with I*K = 10^8 fixed, a tenth
    # of the K coordinates non-empty with 1000 entries each in A (column k) and in B (row k); K swept
    "sweep_first_order": [dict(I=10 ** 8 // K, K=K, J=10 ** 8 // K, live_k=K // 10, per_k=1000) for K in (2500, 5000, 10000, 20000)],
    # Sec. 7.2, second-order workspaces: outer-product SpGEMM, I = K = J = 10^4, the number of non-empty
    # coordinates of the contracted index swept, 1000 entries each
    "sweep_second_order": [dict(I=10 ** 4, K=10 ** 4, J=10 ** 4, live_k=n, per_k=1000) for n in (1, 2, 5, 10, 25, 50, 100, 200, 400, 800, 1600)],
}


def run_sweep(name, args, dev):
    """Dense against sparse workspace over the paper's synthetic shapes; one JSON line."""
    import torch
    from paper_2404_04541_b200 import api, binding
    from workloads import crossover_operands

    ctx = api.Context(dev)
    second = name == "sweep_second_order"
    flush = torch.empty(512 << 20, dtype=torch.uint8, device=dev)
    points = []
    for pt in SWEEPS[name]:
        At, B = crossover_operands(pt["I"], pt["K"], pt["J"], pt["live_k"], pt["per_k"], args.seed)
        dB = api.DeviceCSR.from_host(B, device=dev)
        dA = api.DeviceCSR.from_host(At if second else At.transpose(), device=dev)
        row = dict(pt)
        for policy in ("dense", "ism", "auto"):
            plan = ctx.plan(api.EXPR_OUTER if second else api.EXPR_SPGEMM, (binding.SPWS_CSR,) * 3, np.float64, policy)
            sym = ctx.outer_symbolic if second else ctx.spgemm_symbolic
            try:
                c, state = sym(plan, dA, dB)
                nnzC = c.n[1]
                crd = torch.empty(nnzC, dtype=torch.int32, device=dev)
                val = torch.empty(nnzC, dtype=torch.float64, device=dev)
                times = []
                for s in range(1 + args.steps):
                    flush.fill_(s & 0xff)
                    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
                    e0.record()
                    cc, st = sym(plan, dA, dB)
                    ctx.spgemm_numeric(plan, cc, st, crd=crd, val=val)
                    e1.record()
                    torch.cuda.synchronize()
                    if s > 0:
                        times.append(e0.elapsed_time(e1))
                stats = plan.get_stats()
                row["products"], row["nnzC"] = stats["products"], int(nnzC)
                row[policy + "_ms"] = float(np.mean(times))
                del crd, val
            except binding.SpwsError as exc:
                row[policy + "_ms"] = None
                row[policy + "_error"] = binding.status_string(exc.status)
            plan.close()
        if row.get("dense_ms") and row.get("ism_ms"):
            row["dense_over_sparse"] = row["dense_ms"] / row["ism_ms"]
        points.append(row)
        ctx._scratch = None
        torch.cuda.empty_cache()
    ratios = [p["dense_over_sparse"] for p in points if "dense_over_sparse" in p]
    line = {"metric": "dense_vs_sparse_workspace_time_ratio", "unit": "ratio (dense ms / sparse ms)", "workload": name,
            "value": None, "steps": args.steps, "dtype": "f64", "data": "synthetic", "points": points,
            "sparse_faster_by_up_to": (max(ratios) if ratios else None),
            "dense_faster_by_up_to": (1.0 / min(ratios) if ratios else None),
            "paper_context": "sequential CPU code: sparse workspace up to 27.12x faster than dense, dense up to 7.58x faster than sparse"}
    print(json.dumps(line), flush=True)


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--workload", default="rmat18",
                    help="rmat18 (default), stencil64, uniform8, wide26, ttm4096, rmatNN / stencilNN at another size, "
                         "or sweep_first_order / sweep_second_order (dense against sparse workspace, Sec. 7.2 shapes)")
    ap.add_argument("--policy", default="auto")
    ap.add_argument("--impl", default="spws", choices=["spws", "reference"])
    ap.add_argument("--seed", type=int, default=1)
    ap.add_argument("--opt", action="append", default=[], help="plan option as name=value (repeatable)")
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-targets", action="store_true", help="skip the second target configuration (stencil64)")
    ap.add_argument("--cpu-seconds", type=float, default=12.0, help="CPU time of the oracle sample")
    args = ap.parse_args()
    WORKLOAD_TEXT.setdefault(args.workload, f"{args.workload} (same recipe as the named configuration, other size), fp64")
    if args.impl == "reference":
        run_reference(args)
        return
    if args.warmup < 3:
        args.warmup = 3

    import torch
    import torch.distributed as dist

    world = int(os.environ.get("WORLD_SIZE", "1"))
    rank = int(os.environ.get("RANK", "0"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    torch.cuda.set_device(local)
    dev = torch.device("cuda", local)
    if args.workload in SWEEPS:
        if rank == 0:
            run_sweep(args.workload, args, dev)
        return
    if world > 1:
        dist.init_process_group("nccl", device_id=dev)

    m = measure(args.workload, args, dev, rank, world, dist, e2e=not args.no_e2e, cpu_baseline=not args.no_cpu_baseline)
    line = {"metric": METRIC, "value": m.pop("value"), "unit": UNIT, "n_gpus": world, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": m.pop("ms_per_step"), "higher_is_better": True, "scaling": m.pop("scaling"),
            "vs_baseline": None, "dtype": m.pop("dtype"), "data": "synthetic", "config": m.pop("config")}
    line.update(m)
    # the other configuration with a roofline target, same protocol (default run only)
    if args.workload == "rmat18" and not args.no_targets and not args.opt and args.policy == "auto":
        torch.cuda.empty_cache()
        t = measure("stencil64", args, dev, rank, world, dist, e2e=False, cpu_baseline=False)
        line["targets"] = {"stencil64": {"metric": METRIC, "unit": UNIT, **t}}

    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


if __name__ == "__main__":
    main()
