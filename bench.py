#!/usr/bin/env python
"""Benchmark of the local sparse SYRK path: one JSON line per run.

A step is one pass of the whole hot path over one matrix: plan (transpose, work estimate,
binning), symbolic (count + scan), numeric, mirror, and the Jaccard normalisation when the
matrix is int32.  The default workload is the large Erdos-Renyi configuration (the one the
roofline target is quoted on).  `--impl reference` times the CPU oracle on a bounded sample
of the same workload instead.

  python bench.py [--gpus N] [--steps K] [--warmup W] [--workload 1..5] [--impl ours|reference]

Under torchrun (N > 1) every rank runs an independent replica of the step on its own GPU
(the path does not shard: no collective on the data path); value = N * work / max-over-ranks time.
"""
from __future__ import annotations

import argparse
import json
import os
import subprocess
import sys
import threading
import time

import numpy as np

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

from paper_2608_09713_b200 import workloads as W  # noqa: E402

METRIC = "tril_syrk_useful_multiply_adds_per_s"
UNIT = "MAC/s"
# DRAM bytes per launch of the dominant kernel from the ncu capture summarised under profiles/
# (bytes per useful multiply-add, multiplied by the launch's multiply-adds); None = not captured.
NCU_TRAFFIC_BYTES_PER_MAC = 32.8


def measured_peaks():
    path = os.path.join(ROOT, "MEASURED_PEAKS.json")
    if os.path.exists(path):
        try:
            return float(json.load(open(path))["hbm_gbs"]), "measured"
        except Exception:
            pass
    return 6650.0, "fallback"


class ClockSampler:
    """Samples SM clocks and throttle reasons with nvidia-smi while the timed region runs."""

    Q = ("clocks.sm,clocks.max.sm,clocks_event_reasons.hw_slowdown,clocks_event_reasons.hw_thermal_slowdown,"
         "clocks_event_reasons.sw_thermal_slowdown,clocks_event_reasons.sw_power_cap")

    def __init__(self, index: int):
        self.index, self.samples, self.proc = index, [], None

    def start(self):
        try:
            self.proc = subprocess.Popen(["nvidia-smi", f"--query-gpu={self.Q}", "--format=csv,noheader,nounits",
                                          "-lms", "100", "-i", str(self.index)], stdout=subprocess.PIPE, text=True)
            threading.Thread(target=self._read, daemon=True).start()
        except Exception:
            self.proc = None

    def _read(self):
        for line in self.proc.stdout:
            self.samples.append((time.time(), line.strip()))

    def stop(self, t0, t1):
        if self.proc is None:
            return {"sm_mhz": None, "sm_max_mhz": None, "reasons": ["nvidia-smi unavailable"]}
        time.sleep(0.25)
        self.proc.terminate()
        rows = [s for t, s in self.samples if t0 - 0.05 <= t <= t1 + 0.15] or [s for _, s in self.samples]
        mhz, mx, reasons = [], None, set()
        names = ["hw_slowdown", "hw_thermal_slowdown", "sw_thermal_slowdown", "sw_power_cap"]
        for r in rows:
            f = [x.strip() for x in r.split(",")]
            try:
                mhz.append(float(f[0])); mx = float(f[1])
            except Exception:
                continue
            for nm, v in zip(names, f[2:6]):
                if v.lower().startswith("active"):
                    reasons.add(nm)
        return {"sm_mhz": float(np.median(mhz)) if mhz else None, "sm_max_mhz": mx, "reasons": sorted(reasons),
                "samples": len(mhz)}


def max_over_ranks(x: float, device="cpu") -> float:
    """Maximum of a per-rank number over all ranks (the job is as slow as its slowest replica)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.MAX)
    return float(t.item())


def sum_over_ranks(x: float, device="cpu") -> float:
    """Sum of a per-rank number over all ranks (row-sharded runs: every rank does a part of one job)."""
    import torch
    import torch.distributed as dist
    if not (dist.is_available() and dist.is_initialized()) or dist.get_world_size() == 1:
        return float(x)
    t = torch.tensor([x], dtype=torch.float64, device=device)
    dist.all_reduce(t, op=dist.ReduceOp.SUM)
    return float(t.item())


def whole_job_rate(units_per_rank: float, world: int, ms_per_step: float) -> float:
    """Replicas: every rank processes `units_per_rank` per step; the job's rate counts all of them."""
    return world * units_per_rank / (ms_per_step / 1e3)


def class_of_rows(light_work, deg, work):
    """The library's row classes, recomputed on the host for the roofline's byte counts: light rows (at most 32
    nonzeros) are classed by `light_work` (their products without the diagonal ones in lower-triangle mode)."""
    cls = np.full(work.shape, 7, dtype=np.int8)
    cls[work <= 32768] = 6
    light = (deg <= 32) & (light_work <= 512)
    for c, hi in ((5, 512), (4, 256), (3, 128), (2, 64), (1, 32)):
        cls[light & (light_work <= hi)] = c
    cls[work == 0] = 0
    return cls


def algorithmic_bytes(deg, work, cnt, sv):
    """Bytes the row-by-row method must move for a set of rows: per row of A 8 + d_i (4 + sv) read,
    per multiply-add one (row id, value) entry of a column list read, per output nonzero one
    (column id, value) written, per output row an 8-byte row pointer."""
    return int((8 + deg * (4 + sv)).sum() + work.sum() * (4 + sv) + cnt.sum() * (4 + sv) + 8 * deg.size)


def oracle_sample(a, steps, warmup, budget_s=None):
    """Times the CPU oracle on a contiguous block of rows from the middle of the matrix."""
    import oracle
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, a.vals)
    # size the block for a few seconds of work: probe 1/512 of the rows first
    r0 = a.m // 2
    probe = max(1, a.m // 512)
    t = time.perf_counter()
    res = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, r0, min(a.m, r0 + probe), cols=cols)
    dt = max(time.perf_counter() - t, 1e-6)
    rate = max(float(res.work.sum()), 1.0) / dt
    per_row = max(float(res.work.sum()) / probe, 1.0)
    if budget_s is None:
        budget_s = 20.0 / max(steps + warmup, 1) if (steps + warmup) > 2 else 10.0
    rows = int(min(a.m - r0, max(probe, rate * budget_s / per_row)))
    times, macs, nnz = [], 0, 0
    for it in range(warmup + steps):
        t = time.perf_counter()
        res = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, a.vals, oracle.TRIL, r0, r0 + rows, cols=cols)
        dt = time.perf_counter() - t
        if it >= warmup:
            times.append(dt)
        macs, nnz = int(res.work.sum()), res.nnz
    return {"rows": rows, "r0": r0, "macs": macs, "nnz": nnz, "times": times}


def run_reference(args):
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return
    a = W.config(args.workload)
    s = oracle_sample(a, args.steps, args.warmup)
    ms = 1e3 * float(np.mean(s["times"]))
    value = s["macs"] / (ms / 1e3)
    sample = f"rows [{s['r0']}, {s['r0'] + s['rows']}) of {a.name}: {s['macs']} multiply-adds, {s['nnz']} output nonzeros per step"
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus, "steps": args.steps,
            "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True, "scaling": "weak", "vs_baseline": None,
            "dtype": "f64" if a.vals.dtype == np.float64 else ("f32" if a.vals.dtype == np.float32 else "i32"),
            "data": "synthetic", "config": {"workload": a.name, "sample": sample},
            "nnz_per_s": s["nnz"] / (ms / 1e3),
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle", "sample": sample},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0}}
    print(json.dumps(line), flush=True)


def stats(xs):
    """mean, median and best of a list of per-step milliseconds."""
    xs = [float(x) for x in xs]
    return {"mean": float(np.mean(xs)), "median": float(np.median(xs)), "best": float(np.min(xs))}


def verify_rows(a, c_dev, rows, tol):
    """Rows `rows` of the device result (c_rowptr, c_colidx, c_vals) against the CPU oracle, element by element:
    structure exact, integer values exact, floating-point values within tol * sum |partial products|."""
    import oracle
    rowptr = c_dev[0].cpu().numpy()
    vals64 = np.ascontiguousarray(a.vals, dtype=np.float64)
    cols = oracle.transpose(a.m, a.n, a.rowptr, a.colidx, vals64)
    worst = 0.0
    for r in rows:
        r = int(r)
        ref = oracle.syrk(a.m, a.n, a.rowptr, a.colidx, vals64, oracle.TRIL, r, r + 1, cols=cols)
        lo, hi = int(rowptr[r]), int(rowptr[r + 1])
        if hi - lo != ref.nnz or not np.array_equal(c_dev[1][lo:hi].cpu().numpy(), ref.colidx):
            return False, worst
        got = c_dev[2][lo:hi].cpu().numpy()
        if np.issubdtype(a.vals.dtype, np.integer):
            if not np.array_equal(got, oracle.to_int32(ref.vals)):
                return False, worst
        elif ref.nnz:
            err = np.abs(got.astype(np.float64) - ref.vals) / np.maximum(ref.absvals, 1e-300)
            worst = max(worst, float(err.max()))
            if worst > tol:
                return False, worst
    return True, worst


def measure_workload(a, args, steps, warmup, world, rank, local, headline, dist=None, shard=False):
    """Times `steps` passes of the whole path over one matrix (after `warmup` untimed ones) and returns the
    numbers of that workload: phases, per-class launches, roofline of the dominant numeric launch, the numeric
    pass under both byte models, the mirror, and the full-output variant of the same kernels."""
    import torch
    from paper_2608_09713_b200 import binding as B

    sv = a.vals.dtype.itemsize
    dname = {np.dtype(np.float64): "f64", np.dtype(np.float32): "f32", np.dtype(np.int32): "i32"}[a.vals.dtype]
    is_int = a.vals.dtype == np.int32
    do_mirror = not (args.no_mirror or is_int or shard)  # the 1e5 x 1e5 dense mirror of the binary workload is not asked for
    stream = torch.cuda.current_stream()
    r0, r1, allgather_ms = 0, a.m, None
    if shard:
        # Row-sharded run of ONE product: every rank starts with a slice of A's rows, the slices are
        # all-gathered over NCCL into each GPU's own memory, then each rank computes a range of output rows
        # of near-equal work.  No collective follows on the data path.
        from paper_2608_09713_b200 import sharding as S
        sb = S.row_slice_bounds(a.m, world)
        s0, s1 = sb[rank], sb[rank + 1]
        loc = (torch.from_numpy(a.rowptr[s0:s1 + 1] - a.rowptr[s0]).cuda(), torch.from_numpy(a.colidx[a.rowptr[s0]:a.rowptr[s1]]).cuda(),
               torch.from_numpy(a.vals[a.rowptr[s0]:a.rowptr[s1]]).cuda())
        for it in range(2):
            dist.barrier()
            torch.cuda.synchronize()
            e0 = torch.cuda.Event(enable_timing=True); e1 = torch.cuda.Event(enable_timing=True)
            e0.record(stream)
            d_rowptr, d_colidx, d_vals = S.allgather_csr(a.m, *loc)
            e1.record(stream)
            torch.cuda.synchronize()
            allgather_ms = max_over_ranks(e0.elapsed_time(e1), "cuda")
        del loc
        p0 = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.TRIL)
        r0, r1 = S.rank_rows(B.spsyrk_plan_partition(p0, world), rank)
        del p0
    else:
        d_rowptr, d_colidx, d_vals = (torch.from_numpy(x).cuda() for x in (a.rowptr, a.colidx, a.vals))

    def ev():
        e = torch.cuda.Event(enable_timing=True)
        e.record(stream)
        return e

    # Device buffers are allocated once (sizes come from an untimed sizing pass) and reused by every
    # step, so that no allocator call sits inside the timed region.
    sizing = B.tril_syrk(a.m, a.n, d_rowptr, d_colidx, d_vals, row_begin=r0, row_end=r1)
    nnz0 = sizing[1].numel()
    del sizing
    torch.cuda.empty_cache()
    plan_ws_bytes = B.spsyrk_plan_workspace_bytes(a.m, a.n, a.nnz, d_vals.dtype)
    buf = {"plan_ws": torch.empty(plan_ws_bytes, dtype=torch.uint8, device="cuda"),
           "c_rowptr": torch.empty(a.m + 1, dtype=torch.int64, device="cuda"),
           "c_colidx": torch.empty(max(nnz0, 1), dtype=torch.int32, device="cuda"),
           "c_vals": torch.empty(max(nnz0, 1), dtype=d_vals.dtype, device="cuda")}
    mirror_ws_bytes = 0
    if do_mirror:
        nnz_f0 = 2 * nnz0  # upper bound of nnz(F)
        mirror_ws_bytes = B.spsyrk_mirror_workspace_bytes(a.m, nnz0, d_vals.dtype)
        buf["mirror_ws"] = torch.empty(mirror_ws_bytes, dtype=torch.uint8, device="cuda")
        buf["f"] = (torch.empty(a.m + 1, dtype=torch.int64, device="cuda"), torch.empty(nnz_f0, dtype=torch.int32, device="cuda"),
                    torch.empty(nnz_f0, dtype=d_vals.dtype, device="cuda"))
        if sv == 8:
            B.spsyrk_mirror_enable_timing(True)
    if is_int:
        buf["jac"] = torch.empty(max(nnz0, 1), dtype=torch.float32, device="cuda")
    map_bytes = 0
    if not args.no_map:
        p0 = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.TRIL, row_begin=r0, row_end=r1, workspace=buf["plan_ws"])
        map_bytes = B.spsyrk_plan_map_bytes(p0)
        buf["map"] = torch.empty(max(map_bytes, 256), dtype=torch.uint8, device="cuda")
        del p0

    def step(timing=False, keep=False):
        marks = [ev()]
        plan = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.TRIL, workspace=buf["plan_ws"])
        if timing:
            B.spsyrk_plan_enable_timing(plan)
        if shard:
            B.spsyrk_plan_set_rows(plan, *S.rank_rows(B.spsyrk_plan_partition(plan, world), rank))
        if "map" in buf:
            B.spsyrk_plan_lend_map(plan, buf["map"])
        if is_int and not args.separate_jaccard:
            B.spsyrk_plan_set_jaccard(plan, buf["jac"])  # the numeric pass writes the similarities with the counts
        marks.append(ev())
        c_rowptr, c_colidx, c_vals = buf["c_rowptr"], buf["c_colidx"], buf["c_vals"]
        nnz = B.spsyrk_symbolic(plan, c_rowptr)
        assert nnz == nnz0
        marks.append(ev())
        B.spsyrk_numeric(plan, c_rowptr, c_colidx, c_vals)
        marks.append(ev())
        nnz_f = 0
        mirror_pass_ms = None
        if do_mirror:
            f = B.spsyrk_mirror(a.m, c_rowptr, c_colidx[:nnz], c_vals[:nnz], workspace=buf["mirror_ws"], out=buf["f"])
            nnz_f = f[1].numel()
        marks.append(ev())
        if is_int and args.separate_jaccard:
            B.spsyrk_jaccard(a.m, 0, a.m, d_rowptr, c_rowptr, c_colidx[:nnz], c_vals[:nnz], out=buf["jac"])
        marks.append(ev())
        if do_mirror and sv == 8 and timing:
            mirror_pass_ms = B.spsyrk_mirror_timings()
        out = {"marks": marks, "nnz": nnz, "nnz_full": nnz_f, "plan": plan, "mirror_pass_ms": mirror_pass_ms}
        if keep:
            out["c"] = (c_rowptr, c_colidx[:nnz], c_vals[:nnz])
        return out

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    # ---- the bench's own output against the oracle, before any timing counts (rank 0)
    verified = None
    if rank == 0 and not args.no_verify and not shard:
        chk = step(keep=True)
        torch.cuda.synchronize()
        rng = np.random.default_rng(12345)
        deg = np.diff(a.rowptr)
        if a.m <= 4096:
            rows = np.arange(a.m)
        else:
            # 32 uniform rows, the last row, and the 8 rows of A with the most nonzeros
            rows = np.unique(np.concatenate([rng.integers(0, a.m, size=32), [a.m - 1], np.argsort(deg)[-8:]]))
        tol = 1e-12 if a.vals.dtype == np.float64 else 1e-5
        ok, worst = verify_rows(a, chk["c"], rows, tol)
        verified = {"ok": bool(ok), "rows": int(rows.size), "max_scaled_error": worst, "tolerance": 0.0 if is_int else tol}
        assert ok, f"bench output differs from the oracle on {a.name}: {verified}"
        del chk

    for _ in range(max(warmup, 1)):
        r = step()
        torch.cuda.synchronize()
        del r
    launches0 = B.spsyrk_launch_count()
    sampler = ClockSampler(local)
    if rank == 0:
        sampler.start()
        time.sleep(0.3)
    barrier()
    t0 = time.time()
    results = [step(timing=True) for _ in range(steps)]
    barrier()
    t1 = time.time()
    launches = (B.spsyrk_launch_count() - launches0) // steps
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    total_ms = results[0]["marks"][0].elapsed_time(results[-1]["marks"][-1])
    ms_per_step = max_over_ranks(total_ms / steps, "cuda")
    names = ["plan", "symbolic", "numeric", "mirror", "jaccard"]
    per_step = {nm: [r["marks"][i].elapsed_time(r["marks"][i + 1]) for r in results] for i, nm in enumerate(names)}
    phases = {nm: float(np.mean(v)) for nm, v in per_step.items()}
    step_ms = [r["marks"][0].elapsed_time(r["marks"][-1]) for r in results]
    work_total, class_rows = B.spsyrk_plan_stats(results[-1]["plan"])
    nnz_c, nnz_f = results[-1]["nnz"], results[-1]["nnz_full"]
    sym_ms = np.mean([B.spsyrk_plan_timings(r["plan"])[0] for r in results], axis=0)
    num_ms = np.mean([B.spsyrk_plan_timings(r["plan"])[1] for r in results], axis=0)
    if shard:
        work_total = int(sum_over_ranks(work_total, "cuda"))
        nnz_c = int(sum_over_ranks(nnz_c, "cuda"))
        value = whole_job_rate(work_total, 1, ms_per_step)
    else:
        value = whole_job_rate(work_total, world, ms_per_step)

    out = {"value": value, "ms_per_step": ms_per_step, "dtype": dname, "scaling": "strong" if shard else "weak",
           "config": {"workload": a.name, "m": a.m, "n": a.n, "nnz_a": a.nnz, "multiply_adds": work_total, "nnz_c_l": nnz_c,
                      "nnz_full": nnz_f, "step": "plan+symbolic+numeric" + ("+mirror" if do_mirror else "") + (("+jaccard" if args.separate_jaccard else " (Jaccard fused into numeric)") if is_int else ""),
                      "l2_policy": "inputs_larger_than_l2" if a.nnz * (4 + sv) + nnz_c * (4 + sv) > 126e6 else "l2_flushed_by_the_other_phases",
                      "item_map": "map" in buf, "parallelism": f"rows x{world}" if shard else f"replicas x{world}"},
           "nnz_per_s": whole_job_rate(nnz_c, 1 if shard else world, ms_per_step), "phases_ms": phases,
           "step_ms": stats(step_ms), "phases_ms_median": {nm: float(np.median(v)) for nm, v in per_step.items()},
           "phases_ms_best": {nm: float(np.min(v)) for nm, v in per_step.items()},
           "numeric_class_ms": [float(x) for x in num_ms], "symbolic_class_ms": [float(x) for x in sym_ms],
           "class_rows": class_rows, "gpu_launches": int(launches), "clocks": clocks, "verified": verified,
           "workspace": {"plan_bytes": int(plan_ws_bytes), "plan_over_a": plan_ws_bytes / max(a.rowptr.nbytes + a.colidx.nbytes + a.vals.nbytes, 1),
                         "item_map_bytes": int(map_bytes), "mirror_bytes": int(mirror_ws_bytes),
                         "mirror_over_c_l": mirror_ws_bytes / max(nnz_c * (4 + sv) + 8 * (a.m + 1), 1) if do_mirror else None}}
    if shard:
        out["allgather_ms"] = allgather_ms
        return out, None
    ctx = {"B": B, "buf": buf, "step": step, "ev": ev, "results": results, "d": (d_rowptr, d_colidx, d_vals), "barrier": barrier,
           "num_ms": num_ms, "phases": phases, "per_step": per_step, "nnz_c": nnz_c, "nnz_f": nnz_f, "work_total": work_total,
           "do_mirror": do_mirror, "is_int": is_int, "sv": sv}
    if rank == 0 and not args.skip_extras:
        roofline_and_variants(a, args, out, ctx, headline)
    return out, ctx


def roofline_and_variants(a, args, line, ctx, headline):
    """Roofline of the dominant numeric launch, the numeric pass under both byte models, the mirror and its
    sorting pass, the full-output variant; for the headline workload also the other consumers and forms."""
    import torch
    B, buf, step, ev, results = ctx["B"], ctx["buf"], ctx["step"], ctx["ev"], ctx["results"]
    d_rowptr, d_colidx, d_vals = ctx["d"]
    num_ms, phases, nnz_c, nnz_f, sv, is_int = ctx["num_ms"], ctx["phases"], ctx["nnz_c"], ctx["nnz_f"], ctx["sv"], ctx["is_int"]
    peak, peak_kind = measured_peaks()
    plan = results[-1]["plan"]
    _, _, _, work_dev = B.spsyrk_plan_buffers(plan)
    work = work_dev.cpu().numpy()
    keep = step(keep=True)
    torch.cuda.synchronize()
    cnt = np.diff(keep["c"][0].cpu().numpy())
    deg = np.diff(a.rowptr)
    diag_apart = True  # lower-triangle mode over the whole column range: light rows are classed without their diagonal products
    cls = class_of_rows(work - (deg if diag_apart else 0), deg, work)
    dom = int(np.argmax(num_ms))
    sel = cls == dom
    # Column lists that fit in L2 are read from DRAM once, not once per multiply-add: the launch's
    # algorithmic bytes are then its rows of A, the column lists once, and its output.
    at_bytes = a.nnz * (4 + sv)
    lists_in_l2 = at_bytes < 100e6
    if lists_in_l2:
        bytes_dom = int((8 + deg[sel] * (4 + sv)).sum() + at_bytes + cnt[sel].sum() * (4 + sv) + 8 * int(sel.sum()))
    else:
        bytes_dom = algorithmic_bytes(deg[sel], work[sel], cnt[sel], sv)
    ach = bytes_dom / (num_ms[dom] / 1e3) / 1e9
    if dom <= 5:
        kernel = ("numeric_map_warp_kernel<N=%d>" if line["config"]["item_map"] else "numeric_warp_kernel<N=%d>") % (16 << dom)
    else:
        kernel = "rows_cta_kernel<%d threads, numeric>" % (256 if dom == 6 else 1024)
    traffic = None
    if NCU_TRAFFIC_BYTES_PER_MAC is not None and dom == 4 and a.vals.dtype == np.float64 and not lists_in_l2 and line["config"]["item_map"]:
        traffic = NCU_TRAFFIC_BYTES_PER_MAC * float(work[sel].sum())
    # the every-array-once floor of the same launch: its rows of A, its share of the column lists, its output
    bytes_min_dom = int((8 + deg[sel] * (4 + sv)).sum() + at_bytes * (work[sel].sum() / max(work.sum(), 1)) + cnt[sel].sum() * (4 + sv) + 8 * int(sel.sum()))
    line["roofline"] = {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                        "traffic": traffic, "traffic_kind": "extrapolated from the ncu capture of the same kernel on the 2^20-row copy (bytes per multiply-add x multiply-adds of the launch)" if traffic else None,
                        "peak_kind": peak_kind, "algorithmic_bytes_per_launch": bytes_dom,
                        "bytes_model": "column lists once (L2-resident)" if lists_in_l2 else "one column-list entry per multiply-add (column lists far beyond L2, random columns)",
                        "frac_every_array_once": bytes_min_dom / (num_ms[dom] / 1e3) / 1e9 / peak,
                        "launch_ms": float(num_ms[dom]), "rows_in_launch": int(sel.sum()),
                        "multiply_adds_in_launch": int(work[sel].sum())}
    b_gust = algorithmic_bytes(deg, work, cnt, sv)
    b_min = a.rowptr.nbytes + a.colidx.nbytes + a.vals.nbytes + 8 * (a.n + 1) + a.nnz * (4 + sv) + 8 * (a.m + 1) + nnz_c * (4 + sv)
    num = ctx["per_step"]["numeric"]
    b_rule = b_min if lists_in_l2 else b_gust
    line["numeric_pass"] = {"ms": phases["numeric"], "ms_median": float(np.median(num)), "ms_best": float(np.min(num)),
                            "b_gust_bytes": b_gust, "b_min_bytes": int(b_min),
                            "bytes_rule": "every array once (column lists L2-resident)" if lists_in_l2 else "one column-list entry per multiply-add",
                            "gbs": b_rule / (phases["numeric"] / 1e3) / 1e9, "frac_of_peak": b_rule / (phases["numeric"] / 1e3) / 1e9 / peak,
                            "frac_of_peak_b_gust": b_gust / (phases["numeric"] / 1e3) / 1e9 / peak,
                            "frac_of_peak_every_array_once": b_min / (phases["numeric"] / 1e3) / 1e9 / peak,
                            "frac_of_8tbs": b_rule / (phases["numeric"] / 1e3) / 1e9 / 8000.0}
    if ctx["do_mirror"]:
        mb = nnz_c * (4 + sv) + 8 * (a.m + 1) + nnz_f * (4 + sv) + 8 * (a.m + 1)
        mir = ctx["per_step"]["mirror"]
        line["mirror_pass"] = {"ms": phases["mirror"], "ms_median": float(np.median(mir)), "ms_best": float(np.min(mir)), "bytes": int(mb),
                               "gbs": mb / (phases["mirror"] / 1e3) / 1e9, "frac_of_peak": mb / (phases["mirror"] / 1e3) / 1e9 / peak}
        pms = [r["mirror_pass_ms"] for r in results if r["mirror_pass_ms"]]
        if pms:
            pm = np.mean(np.array(pms), axis=0)
            # one sorting pass moves a 16-byte record in and out plus the digit byte it writes and the next histogram reads
            pass_bytes = nnz_c * (16 + 16 + 2)
            mid = int(np.argmax(pm))
            line["mirror_pass"]["sort_passes_ms"] = [float(x) for x in pm]
            line["mirror_pass"]["sort_pass_roofline"] = {"bound": "hbm", "kernel": "mirror_pass_kernel (histogram + scan + scatter of one pass)",
                                                         "bytes_per_pass": int(pass_bytes), "achieved": pass_bytes / (float(pm[mid]) / 1e3) / 1e9,
                                                         "peak": peak, "unit": "GB/s", "frac": pass_bytes / (float(pm[mid]) / 1e3) / 1e9 / peak}
    if not headline:
        del keep
        full_variant(a, args, line, ctx)
        one_pass_variant(a, args, line, ctx)
        return
    # ---- consuming the triangle directly: y = C_L x + C_L^T x - D x and Y = C X (floating-point workloads)
    if not is_int:
        xv = torch.ones(a.m, dtype=d_vals.dtype, device="cuda")
        yv = torch.empty_like(xv)
        st_ = []
        for it in range(4):
            e0 = ev()
            B.spsyrk_symv(a.m, keep["c"][0], keep["c"][1], keep["c"][2], xv, yv)
            e1 = ev()
            torch.cuda.synchronize()
            st_.append(e0.elapsed_time(e1))
        sb = nnz_c * (4 + sv) + 8 * (a.m + 1) + 2 * a.m * sv
        sm = float(np.mean(st_[1:]))
        line["symv"] = {"ms": sm, "bytes": int(sb), "gbs": sb / (sm / 1e3) / 1e9, "frac_of_peak": sb / (sm / 1e3) / 1e9 / peak}
        if not args.no_verify:
            # whole-matrix check that needs no oracle: C_L x + C_L^T x - D x must equal A (A^T x) for a random x
            # (Section V-F); the right-hand side from plain tensor operations on A, in double
            gen = torch.Generator(device="cuda")
            gen.manual_seed(20260807)
            x64 = torch.rand(a.m, dtype=torch.float64, device="cuda", generator=gen) - 0.5
            B.spsyrk_symv(a.m, keep["c"][0], keep["c"][1], keep["c"][2], x64.to(d_vals.dtype), yv)
            xq = x64.to(d_vals.dtype).double()   # the vector the kernel saw
            rows = torch.repeat_interleave(torch.arange(a.m, device="cuda"), d_rowptr[1:] - d_rowptr[:-1])
            cols = d_colidx.long()
            v64 = d_vals.double()
            z = torch.zeros(a.n, dtype=torch.float64, device="cuda").index_add_(0, cols, v64 * xq[rows])
            y_ref = torch.zeros(a.m, dtype=torch.float64, device="cuda").index_add_(0, rows, v64 * z[cols])
            za = torch.zeros(a.n, dtype=torch.float64, device="cuda").index_add_(0, cols, v64.abs() * xq[rows].abs())
            scale = torch.zeros(a.m, dtype=torch.float64, device="cuda").index_add_(0, rows, v64.abs() * za[cols])
            worst = float(((yv.double() - y_ref).abs() / scale.clamp_min(1e-300)).max())
            tol = 1e-12 if sv == 8 else 1e-5
            line["symv"]["identity_with_A_At_x"] = {"max_scaled_error": worst, "tolerance": tol, "ok": bool(worst <= tol)}
            del x64, xq, rows, cols, v64, z, y_ref, za, scale
        del xv, yv
        pcols = 8
        xm = torch.ones((a.m, pcols), dtype=d_vals.dtype, device="cuda")
        ym = torch.empty_like(xm)
        st_ = []
        for it in range(4):
            e0 = ev()
            B.spsyrk_symm(a.m, keep["c"][0], keep["c"][1], keep["c"][2], xm, ym)
            e1 = ev()
            torch.cuda.synchronize()
            st_.append(e0.elapsed_time(e1))
        sb = nnz_c * (4 + sv) + 8 * (a.m + 1) + 2 * a.m * pcols * sv
        sm = float(np.mean(st_[1:]))
        line["symm"] = {"columns": pcols, "ms": sm, "bytes": int(sb), "gbs": sb / (sm / 1e3) / 1e9, "frac_of_peak": sb / (sm / 1e3) / 1e9 / peak}
        del xm, ym
    # ---- 1-D row sharding study (load balance): symbolic + numeric time of each of 8 contiguous row ranges,
    # cut by equal row counts and by equal work (spsyrk_plan_partition); the slowest range is what a
    # row-distributed run would wait for
    parts = 8
    splan = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.TRIL, workspace=buf["plan_ws"])
    splits = {"equal_work": B.spsyrk_plan_partition(splan, parts), "equal_rows": [a.m * p // parts for p in range(parts + 1)]}
    prefix = np.concatenate([[0], np.cumsum(work)])
    shard = {"parts": parts}
    for nm, bounds in splits.items():
        ms_parts = []
        for p_ in range(parts):
            r0_, r1_ = int(bounds[p_]), int(bounds[p_ + 1])
            if r1_ <= r0_:
                ms_parts.append(0.0)
                continue
            B.spsyrk_plan_set_rows(splan, r0_, r1_)
            if "map" in buf:
                B.spsyrk_plan_lend_map(splan, buf["map"])
            for it in range(2):
                e0 = ev()
                B.spsyrk_symbolic(splan, buf["c_rowptr"])
                B.spsyrk_numeric(splan, buf["c_rowptr"], buf["c_colidx"], buf["c_vals"])
                e1 = ev()
                torch.cuda.synchronize()
            ms_parts.append(e0.elapsed_time(e1))
        share = np.diff(prefix[np.asarray(bounds)]).astype(np.float64)
        shard[nm] = {"work_max_over_mean": float(share.max() / max(share.mean(), 1.0)),
                     "ms_max_over_mean": float(max(ms_parts) / max(np.mean(ms_parts), 1e-9)),
                     "ms_max": float(max(ms_parts)), "ms_sum": float(sum(ms_parts))}
    line["row_sharding"] = shard
    del splan
    if a.m == a.n and not is_int:
        # the symmetric random permutation as a device pre-pass (same map for rows and columns)
        g = torch.Generator(device="cpu").manual_seed(1234)
        pm = torch.randperm(a.m, generator=g).to(torch.int32).cuda()
        for it in range(2):
            torch.cuda.synchronize()
            e0 = ev()
            pb = B.spsyrk_permute(a.m, a.n, d_rowptr, d_colidx, d_vals, pm, pm)
            e1 = ev()
            torch.cuda.synchronize()
            del pb
        line["permute_ms"] = e0.elapsed_time(e1)
        del pm
    del keep
    full_variant(a, args, line, ctx)
    one_pass_variant(a, args, line, ctx)
    if args.no_full:
        return
    # ---- a half-block product of the local computation: rows of the second half against the
    # first half of the rows as output columns (an off-diagonal block), full mode
    bplan = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.FULL)
    h = a.m // 2
    bt = []
    for it in range(3):
        e0 = ev()
        B.spsyrk_plan_set_block(bplan, h, a.m, 0, h)
        e1 = ev()
        brp = torch.empty(a.m - h + 1, dtype=torch.int64, device="cuda")
        bn = B.spsyrk_symbolic(bplan, brp)
        e2 = ev()
        bci = torch.empty(max(bn, 1), dtype=torch.int32, device="cuda")
        bcv = torch.empty(max(bn, 1), dtype=d_vals.dtype, device="cuda")
        B.spsyrk_numeric(bplan, brp, bci, bcv)
        e3 = ev()
        torch.cuda.synchronize()
        bt.append((e0.elapsed_time(e1), e1.elapsed_time(e2), e2.elapsed_time(e3)))
        del brp, bci, bcv
    bw, _ = B.spsyrk_plan_stats(bplan)
    line["block_variant"] = {"block": f"rows [{h}, {a.m}) x columns [0, {h})", "multiply_adds": bw, "nnz": bn,
                             "set_block_ms": float(np.mean([t[0] for t in bt[1:]])),
                             "symbolic_ms": float(np.mean([t[1] for t in bt[1:]])),
                             "numeric_ms": float(np.mean([t[2] for t in bt[1:]]))}
    del bplan
    # ---- the accumulating form: C_L = tril(A_0 A_0^T) + tril(A_1 A_1^T) over two column panels of A
    if nnz_c * (4 + sv) < 20e9:
        pt = []
        for it in range(3):  # the first round also warms the allocator: later rounds reuse its blocks
            e = [ev()]
            prods = []
            for k0, k1 in ((0, a.n // 2), (a.n // 2, a.n)):
                pnl = B.spsyrk_column_panel(a.m, d_rowptr, d_colidx, d_vals, k0, k1)
                e.append(ev())
                t_rp, t_ci, t_cv, _ = B.tril_syrk(a.m, a.n, *pnl)
                e.append(ev())
                prods.append((t_rp, t_ci, t_cv))
            z = B.spsyrk_accumulate(a.m, *prods[0], *prods[1])
            e.append(ev())
            torch.cuda.synchronize()
            pt.append([e[i].elapsed_time(e[i + 1]) for i in range(5)])
            zn = int(z[1].numel())
            ab = sum(int(t[1].numel()) for t in prods) * (4 + sv) + zn * (4 + sv) + 3 * 8 * (a.m + 1)
            del prods, z, pnl, t_rp, t_ci, t_cv
        pm = np.mean(np.array(pt[1:]), axis=0)
        line["panel_variant"] = {"panels": 2, "nnz_sum": zn, "nnz_matches_unsplit": zn == nnz_c,
                                 "column_panel_ms": float(pm[0] + pm[2]), "products_ms": float(pm[1] + pm[3]),
                                 "accumulate_ms": float(pm[4]), "accumulate_bytes": int(ab),
                                 "accumulate_gbs": ab / (float(pm[4]) / 1e3) / 1e9,
                                 "accumulate_frac_of_peak": ab / (float(pm[4]) / 1e3) / 1e9 / peak}
    torch.cuda.empty_cache()


def one_pass_variant(a, args, line, ctx):
    """The one-pass mode (slots sized by the work estimate, counts found while computing, compaction) beside the
    two passes of the timed step: the same C_L, the column lists gathered once."""
    import torch
    B, ev = ctx["B"], ctx["ev"]
    d_rowptr, d_colidx, d_vals = ctx["d"]
    phases, sv, nnz_c = ctx["phases"], ctx["sv"], ctx["nnz_c"]
    if args.no_full:
        return
    if ctx.get("is_int") and not args.separate_jaccard:
        line["one_pass"] = {"skipped": "the timed step writes the similarities with the counts; the one-pass mode does not"}
        return
    if 2.2 * nnz_c * (4 + sv) > 60e9:
        line["one_pass"] = {"skipped": "slot and result buffers together would take about %.0f GB" % (2.2 * nnz_c * (4 + sv) / 1e9)}
        return
    plan = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.TRIL)
    tt = []
    slots = nnz = 0
    for it in range(3):
        e0 = ev()
        slots = B.spsyrk_onepass_slots(plan)
        s_col = torch.empty(max(slots, 1), dtype=torch.int32, device="cuda")
        s_val = torch.empty(max(slots, 1), dtype=d_vals.dtype, device="cuda")
        c_rowptr = torch.empty(a.m + 1, dtype=torch.int64, device="cuda")
        e1 = ev()
        nnz = B.spsyrk_onepass_numeric(plan, s_col, s_val, c_rowptr)
        c_col = torch.empty(max(nnz, 1), dtype=torch.int32, device="cuda")
        c_val = torch.empty(max(nnz, 1), dtype=d_vals.dtype, device="cuda")
        e2 = ev()
        B.spsyrk_onepass_compact(plan, c_rowptr, nnz, s_col, s_val, c_col, c_val)
        e3 = ev()
        torch.cuda.synchronize()
        tt.append((e0.elapsed_time(e1), e1.elapsed_time(e2), e2.elapsed_time(e3)))
        del s_col, s_val, c_rowptr, c_col, c_val
    sl, nu, co = (float(np.mean([t[i] for t in tt[1:]])) for i in (0, 1, 2))
    line["one_pass"] = {"slots_ms": sl, "numeric_ms": nu, "compact_ms": co, "total_ms": sl + nu + co, "four_array_form_ms": sl + nu,
                        "two_pass_ms": phases["symbolic"] + phases["numeric"], "slot_entries": int(slots), "nnz": int(nnz),
                        "slot_entries_over_nnz": slots / max(nnz, 1)}
    assert nnz == nnz_c, "the one-pass mode and the symbolic pass disagree on nnz(C_L)"
    B.spsyrk_destroy(plan)
    torch.cuda.empty_cache()


def full_variant(a, args, line, ctx):
    """The full-output variant of the same kernels (symbolic + numeric only), to show the work the symmetry saves."""
    import torch
    B, buf, ev = ctx["B"], ctx["buf"], ctx["ev"]
    d_rowptr, d_colidx, d_vals = ctx["d"]
    phases, sv, nnz_c = ctx["phases"], ctx["sv"], ctx["nnz_c"]
    f_mirror = buf.pop("f", None); buf.pop("mirror_ws", None)   # F of the last timed step, for the comparison below
    torch.cuda.empty_cache()
    if args.no_full:
        return
    if 2 * nnz_c * (4 + sv) > 60e9:
        line["full_variant"] = {"skipped": "the full product of this workload has about %.0f GB of entries" % (2 * nnz_c * (4 + sv) / 1e9)}
        return
    fplan = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.FULL)
    fmap = torch.empty(max(B.spsyrk_plan_map_bytes(fplan), 256), dtype=torch.uint8, device="cuda") if "map" in buf else None
    if fmap is not None:
        B.spsyrk_plan_lend_map(fplan, fmap)
    fw, _ = B.spsyrk_plan_stats(fplan)
    tt = []
    mirror_check = None
    for it in range(3):
        if it == 1:
            f_mirror = None  # (no cache flush here: the timed iterations reuse the blocks the first one allocated)
        e0 = ev()
        frp = torch.empty(a.m + 1, dtype=torch.int64, device="cuda")
        fn = B.spsyrk_symbolic(fplan, frp)
        e1 = ev()
        fci = torch.empty(max(fn, 1), dtype=torch.int32, device="cuda")
        fcv = torch.empty(max(fn, 1), dtype=d_vals.dtype, device="cuda")
        B.spsyrk_numeric(fplan, frp, fci, fcv)
        e2 = ev()
        torch.cuda.synchronize()
        tt.append((e0.elapsed_time(e1), e1.elapsed_time(e2)))
        if it == 0 and f_mirror is not None and not args.no_verify:
            # the mirrored lower triangle against the full product computed directly: same structure bit for bit,
            # values within the workload's tolerance (the two halves of the full product sum in their own orders)
            same = bool(torch.equal(f_mirror[0], frp)) and bool(torch.equal(f_mirror[1][:fn], fci[:fn]))
            worst = None
            if same and fn > 0:
                x, y = f_mirror[2][:fn], fcv[:fn]
                if x.dtype.is_floating_point:
                    worst = float(((x - y).abs() / torch.maximum(x.abs(), y.abs()).clamp_min(1e-300)).max())
                else:
                    worst = float((x != y).sum())
            mirror_check = {"structure_identical": same, "max_relative_difference_of_values": worst, "entries": int(fn)}
        del frp, fci, fcv
    fs, fnum = (float(np.mean([t[i] for t in tt[1:]])) for i in (0, 1))
    line["full_variant"] = {"multiply_adds": fw, "nnz": fn, "symbolic_ms": fs, "numeric_ms": fnum,
                            "tril_speedup_numeric": fnum / phases["numeric"],
                            "tril_speedup_symbolic_plus_numeric": (fs + fnum) / (phases["symbolic"] + phases["numeric"]),
                            "full_direct_vs_tril_plus_mirror": ((fs + fnum) / (phases["symbolic"] + phases["numeric"] + phases["mirror"])
                                                                if ctx["do_mirror"] else None)}
    if mirror_check is not None:
        line["full_variant"]["mirror_equals_full_product"] = mirror_check
    del fplan, fmap
    torch.cuda.empty_cache()


def run_ours(args):
    import torch
    import torch.distributed as dist
    from paper_2608_09713_b200 import binding as B

    rank = int(os.environ.get("RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    local = int(os.environ.get("LOCAL_RANK", "0"))
    assert torch.cuda.is_available(), "bench.py needs a CUDA device; there is no CPU fallback"
    torch.cuda.set_device(local)
    if world > 1:
        dist.init_process_group("nccl", device_id=torch.device("cuda", local))
    a = W.config(args.workload)
    if args.er_log2m:
        a = W.erdos_renyi(1 << args.er_log2m, 1 << args.er_log2m, 16, W.SEED + 5, np.float64, -1.0, 1.0)
    if args.zipf_rows:
        a = W.zipf_binary(args.zipf_rows, 1 << 22, 100, 1.1, W.SEED + 2)
    if args.rmat_scale:
        a = W.rmat(args.rmat_scale, 16, W.SEED + 3, permute=not args.rmat_noperm)
    shard = bool(args.shard_rows) and world > 1
    res, ctx = measure_workload(a, args, args.steps, args.warmup, world, rank, local, True, dist if world > 1 else None, shard)
    line = {"metric": METRIC, "value": res.pop("value"), "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": res.pop("ms_per_step"), "higher_is_better": True, "scaling": res.pop("scaling"), "vs_baseline": None,
            "dtype": res.pop("dtype"), "data": "synthetic"}
    line.update(res)
    if shard:
        if rank == 0:
            print(json.dumps(line))
        dist.destroy_process_group()
        return
    B_ = ctx["B"]
    work_total, nnz_c, sv = ctx["work_total"], ctx["nnz_c"], ctx["sv"]
    d_dtype = ctx["d"][2].dtype
    ctx["buf"].clear()
    ctx["results"].clear()
    ctx.clear()
    torch.cuda.empty_cache()

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    if not args.skip_extras:
        h_in = tuple(torch.from_numpy(x).pin_memory() for x in (a.rowptr, a.colidx, a.vals))
        out = (torch.empty(a.m + 1, dtype=torch.int64, pin_memory=True), torch.empty(max(nnz_c, 1), dtype=torch.int32, pin_memory=True),
               torch.empty(max(nnz_c, 1), dtype=d_dtype, pin_memory=True))
        B_.spsyrk_host_tril(a.m, a.n, *h_in, out=out)  # warm-up
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        ts = time.perf_counter()
        for _ in range(args.steps):
            B_.spsyrk_host_tril(a.m, a.n, *h_in, out=out)
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()
        e2e_ms = (time.perf_counter() - ts) * 1e3 / args.steps
        e2e_ms = max_over_ranks(e2e_ms, "cuda")
        h2d = a.rowptr.nbytes + a.colidx.nbytes + a.vals.nbytes
        d2h = 8 * (a.m + 1) + nnz_c * (4 + sv)
        line["e2e"] = {"value": whole_job_rate(work_total, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                       "what": "spsyrk_host_tril: H2D of A, plan+symbolic+numeric, D2H of C_L (mirror not included)"}
        del h_in, out
        B_.spsyrk_host_release_cache()
        torch.cuda.empty_cache()

    # ---- the other four workloads, each with its own (shorter) timed run, rank 0 of a 1-GPU run only
    if rank == 0 and world == 1 and not args.skip_extras and not args.no_others and args.workload == 5 and not (
            args.er_log2m or args.zipf_rows or args.rmat_scale):
        others = {}
        for w in (1, 2, 3, 4):
            aw = W.config(w)
            ro, cx = measure_workload(aw, args, max(2, min(args.steps, 3)), 3, 1, 0, local, False)
            if cx is not None:
                cx["buf"].clear(); cx["results"].clear(); cx.clear()
            keep = ("value", "ms_per_step", "dtype", "config", "nnz_per_s", "phases_ms", "phases_ms_median", "step_ms", "class_rows",
                    "numeric_class_ms", "roofline", "numeric_pass", "mirror_pass", "full_variant", "one_pass", "clocks", "verified", "workspace")
            others[f"config_{w}"] = {k: ro[k] for k in keep if k in ro}
            del aw, ro, cx
            B_.spsyrk_host_release_cache()
            torch.cuda.empty_cache()
        line["other_workloads"] = others

    if rank == 0 and world == 1 and not args.skip_extras and not args.no_cpu:
        oracle_sample(a, 1, 0, budget_s=2.0)  # warms the oracle leg (library load, page faults, column lists)
        s = oracle_sample(a, 1, 0)
        line["cpu_baseline"] = {"value": s["macs"] / s["times"][0], "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"rows [{s['r0']}, {s['r0'] + s['rows']}) of {a.name}: {s['macs']} multiply-adds in {s['times'][0]:.2f} s (after one warm-up run)"}
    if rank == 0:
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=5)
    ap.add_argument("--warmup", type=int, default=3)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", type=int, default=5, choices=[1, 2, 3, 4, 5])
    ap.add_argument("--no-mirror", action="store_true")
    ap.add_argument("--no-full", action="store_true")
    ap.add_argument("--no-map", action="store_true", help="do not lend the item map: symbolic counts with hash sets, numeric sorts")
    ap.add_argument("--no-cpu", action="store_true")
    ap.add_argument("--separate-jaccard", action="store_true", help="int32 workloads: Jaccard as its own pass over the counts instead of fused into numeric")
    ap.add_argument("--no-others", action="store_true", help="headline workload only (skip the shorter runs of configurations 1-4)")
    ap.add_argument("--no-verify", action="store_true", help="skip the comparison of sampled output rows with the oracle")
    ap.add_argument("--rmat-noperm", action="store_true", help="with --rmat-scale: skip the random relabelling (load-balance study)")
    ap.add_argument("--shard-rows", action="store_true",
                    help="N > 1 only: one product, output rows split over the ranks by equal work (default: N replicas)")
    ap.add_argument("--skip-extras", action="store_true", help="timed steps only (for profiler runs)")
    ap.add_argument("--zipf-rows", type=int, default=0,
                    help="profiling aid: replace the workload by the binary Zipf recipe with this many rows")
    ap.add_argument("--rmat-scale", type=int, default=0, help="profiling aid: R-MAT recipe at this scale")
    ap.add_argument("--er-log2m", type=int, default=0,
                    help="profiling aid: replace the workload by the large Erdos-Renyi recipe at m = n = 2**k")
    args = ap.parse_args()
    if args.impl == "reference":
        run_reference(args)
    else:
        run_ours(args)


if __name__ == "__main__":
    main()
