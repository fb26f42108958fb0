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
NCU_TRAFFIC_BYTES_PER_MAC = 34.5


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


def class_of_rows(work, deg):
    """The library's row classes, recomputed on the host for the roofline's byte counts."""
    cls = np.full(work.shape, 7, dtype=np.int8)
    cls[work <= 8192] = 6
    light = (deg <= 32) & (work <= 512)
    for c, hi in ((5, 512), (4, 256), (3, 128), (2, 64), (1, 32)):
        cls[light & (work <= hi)] = c
    cls[work == 0] = 0
    return cls


def algorithmic_bytes(deg, work, cnt, sv):
    """Bytes the row-by-row method must move for a set of rows: per row of A 8 + d_i (4 + sv) read,
    per multiply-add one (row id, value) entry of a column list read, per output nonzero one
    (column id, value) written, per output row an 8-byte row pointer."""
    return int((8 + deg * (4 + sv)).sum() + work.sum() * (4 + sv) + cnt.sum() * (4 + sv) + 8 * deg.size)


def oracle_sample(a, steps, warmup):
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
    sv = a.vals.dtype.itemsize
    dname = {np.dtype(np.float64): "f64", np.dtype(np.float32): "f32", np.dtype(np.int32): "i32"}[a.vals.dtype]
    is_int = a.vals.dtype == np.int32
    shard = bool(args.shard_rows) and world > 1
    do_mirror = not (args.no_mirror or is_int or shard)  # the 1e5 x 1e5 dense mirror of config 2 is not asked for
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
    buf = {"plan_ws": torch.empty(B.spsyrk_plan_workspace_bytes(a.m, a.n, a.nnz, d_vals.dtype), dtype=torch.uint8, device="cuda"),
           "c_rowptr": torch.empty(a.m + 1, dtype=torch.int64, device="cuda"),
           "c_colidx": torch.empty(max(nnz0, 1), dtype=torch.int32, device="cuda"),
           "c_vals": torch.empty(max(nnz0, 1), dtype=d_vals.dtype, device="cuda")}
    if do_mirror:
        nnz_f0 = 2 * nnz0  # upper bound of nnz(F)
        buf["mirror_ws"] = torch.empty(B.spsyrk_mirror_workspace_bytes(a.m, nnz0, d_vals.dtype), dtype=torch.uint8, device="cuda")
        buf["f"] = (torch.empty(a.m + 1, dtype=torch.int64, device="cuda"), torch.empty(nnz_f0, dtype=torch.int32, device="cuda"),
                    torch.empty(nnz_f0, dtype=d_vals.dtype, device="cuda"))
    if is_int:
        buf["jac"] = torch.empty(max(nnz0, 1), dtype=torch.float32, device="cuda")
    if not args.no_map:
        p0 = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.TRIL, row_begin=r0, row_end=r1, workspace=buf["plan_ws"])
        buf["map"] = torch.empty(max(B.spsyrk_plan_map_bytes(p0), 256), dtype=torch.uint8, device="cuda")
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
        marks.append(ev())
        c_rowptr, c_colidx, c_vals = buf["c_rowptr"], buf["c_colidx"], buf["c_vals"]
        nnz = B.spsyrk_symbolic(plan, c_rowptr)
        assert nnz == nnz0
        marks.append(ev())
        B.spsyrk_numeric(plan, c_rowptr, c_colidx, c_vals)
        marks.append(ev())
        nnz_f = 0
        if do_mirror:
            f = B.spsyrk_mirror(a.m, c_rowptr, c_colidx[:nnz], c_vals[:nnz], workspace=buf["mirror_ws"], out=buf["f"])
            nnz_f = f[1].numel()
        marks.append(ev())
        if is_int:
            B.spsyrk_jaccard(a.m, 0, a.m, d_rowptr, c_rowptr, c_colidx[:nnz], c_vals[:nnz], out=buf["jac"])
        marks.append(ev())
        out = {"marks": marks, "nnz": nnz, "nnz_full": nnz_f, "plan": plan}
        if keep:
            out["c"] = (c_rowptr, c_colidx[:nnz], c_vals[:nnz])
        return out

    def barrier():
        if world > 1:
            dist.barrier()
        torch.cuda.synchronize()

    for _ in range(max(args.warmup, 1)):
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
    results = [step(timing=True) for _ in range(args.steps)]
    barrier()
    t1 = time.time()
    launches = (B.spsyrk_launch_count() - launches0) // args.steps
    clocks = sampler.stop(t0, t1) if rank == 0 else None
    total_ms = results[0]["marks"][0].elapsed_time(results[-1]["marks"][-1])
    ms_per_step = total_ms / args.steps
    ms_per_step = max_over_ranks(ms_per_step, "cuda")
    names = ["plan", "symbolic", "numeric", "mirror", "jaccard"]
    phases = {nm: float(np.mean([r["marks"][i].elapsed_time(r["marks"][i + 1]) for r in results])) for i, nm in enumerate(names)}
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

    line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps, "warmup": args.warmup,
            "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "strong" if shard else "weak", "vs_baseline": None, "dtype": dname,
            "data": "synthetic",
            "config": {"workload": a.name, "m": a.m, "n": a.n, "nnz_a": a.nnz, "multiply_adds": work_total, "nnz_c_l": nnz_c,
                       "nnz_full": nnz_f, "step": "plan+symbolic+numeric" + ("+mirror" if do_mirror else "") + ("+jaccard" if is_int else ""),
                       "l2_policy": "inputs_larger_than_l2", "parallelism": f"rows x{world}" if shard else f"replicas x{world}"},
            "nnz_per_s": whole_job_rate(nnz_c, 1 if shard else world, ms_per_step), "phases_ms": phases,
            "numeric_class_ms": [float(x) for x in num_ms], "symbolic_class_ms": [float(x) for x in sym_ms],
            "class_rows": class_rows, "gpu_launches": int(launches), "clocks": clocks}

    if shard:
        line["allgather_ms"] = allgather_ms
        if rank == 0:
            print(json.dumps(line))
        dist.destroy_process_group()
        return
    if rank == 0 and not args.skip_extras:
        # ---- roofline of the dominant kernel (the numeric launch of the heaviest row class)
        peak, peak_kind = measured_peaks()
        plan = results[-1]["plan"]
        _, _, _, work_dev = B.spsyrk_plan_buffers(plan)
        work = work_dev.cpu().numpy()
        keep = step(keep=True)
        torch.cuda.synchronize()
        cnt = np.diff(keep["c"][0].cpu().numpy())
        deg = np.diff(a.rowptr)
        cls = class_of_rows(work, deg)
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
        kernel = ("numeric_warp_kernel<N=%d>" % (16 << dom)) if dom <= 5 else ("rows_cta_kernel<%d threads, numeric>" % (256 if dom == 6 else 1024))
        traffic = None
        if NCU_TRAFFIC_BYTES_PER_MAC is not None and dom == 4 and a.vals.dtype == np.float64 and not lists_in_l2:
            traffic = NCU_TRAFFIC_BYTES_PER_MAC * float(work[sel].sum())
        line["roofline"] = {"bound": "hbm", "kernel": kernel, "achieved": ach, "peak": peak, "unit": "GB/s", "frac": ach / peak,
                            "traffic": traffic, "peak_kind": peak_kind, "algorithmic_bytes_per_launch": bytes_dom,
                            "bytes_model": "column lists once (L2-resident)" if lists_in_l2 else "one column-list entry per multiply-add",
                            "launch_ms": float(num_ms[dom]), "rows_in_launch": int(sel.sum()),
                            "multiply_adds_in_launch": int(work[sel].sum())}
        b_gust = algorithmic_bytes(deg, work, cnt, sv)
        b_min = a.rowptr.nbytes + a.colidx.nbytes + a.vals.nbytes + 8 * (a.n + 1) + a.nnz * (4 + sv) + 8 * (a.m + 1) + nnz_c * (4 + sv)
        line["numeric_pass"] = {"ms": phases["numeric"], "b_gust_bytes": b_gust, "b_min_bytes": int(b_min),
                                "gbs_b_gust": b_gust / (phases["numeric"] / 1e3) / 1e9, "frac_of_peak": b_gust / (phases["numeric"] / 1e3) / 1e9 / peak,
                                "frac_of_8tbs": b_gust / (phases["numeric"] / 1e3) / 1e9 / 8000.0}
        if do_mirror:
            mb = nnz_c * (4 + sv) + 8 * (a.m + 1) + nnz_f * (4 + sv) + 8 * (a.m + 1)
            line["mirror_pass"] = {"ms": phases["mirror"], "bytes": int(mb), "gbs": mb / (phases["mirror"] / 1e3) / 1e9,
                                   "frac_of_peak": mb / (phases["mirror"] / 1e3) / 1e9 / peak}
        # ---- consuming the triangle directly: y = C_L x + C_L^T x - D x (floating-point workloads)
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
            del xv, yv
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
        buf.pop("f", None); buf.pop("mirror_ws", None)
        torch.cuda.empty_cache()
        # ---- the full-output variant of the same kernels (symbolic + numeric only)
        if not args.no_full:
            fplan = B.spsyrk_plan(a.m, a.n, d_rowptr, d_colidx, d_vals, mode=B.FULL)
            fw, _ = B.spsyrk_plan_stats(fplan)
            tt = []
            for it in range(3):
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
                del frp, fci, fcv
            fs, fnum = (float(np.mean([t[i] for t in tt[1:]])) for i in (0, 1))
            line["full_variant"] = {"multiply_adds": fw, "nnz": fn, "symbolic_ms": fs, "numeric_ms": fnum,
                                    "tril_speedup_numeric": fnum / phases["numeric"],
                                    "tril_speedup_symbolic_plus_numeric": (fs + fnum) / (phases["symbolic"] + phases["numeric"])}
            del fplan
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

    # ---- end to end through the host-buffer entry point (pinned host memory, copies inside the timed region)
    if not args.skip_extras:
        h_in = tuple(torch.from_numpy(x).pin_memory() for x in (a.rowptr, a.colidx, a.vals))
        out = (torch.empty(a.m + 1, dtype=torch.int64, pin_memory=True), torch.empty(max(nnz_c, 1), dtype=torch.int32, pin_memory=True),
               torch.empty(max(nnz_c, 1), dtype=d_vals.dtype, pin_memory=True))
        del d_rowptr, d_colidx, d_vals, results
        buf.clear()
        torch.cuda.empty_cache()
        B.spsyrk_host_tril(a.m, a.n, *h_in, out=out)  # warm-up
        barrier()
        ts = time.perf_counter()
        for _ in range(args.steps):
            B.spsyrk_host_tril(a.m, a.n, *h_in, out=out)
        barrier()
        e2e_ms = (time.perf_counter() - ts) * 1e3 / args.steps
        e2e_ms = max_over_ranks(e2e_ms, "cuda")
        h2d = a.rowptr.nbytes + a.colidx.nbytes + a.vals.nbytes
        d2h = 8 * (a.m + 1) + nnz_c * (4 + sv)
        line["e2e"] = {"value": whole_job_rate(work_total, world, e2e_ms), "unit": UNIT, "ms_per_step": e2e_ms,
                       "h2d_bytes_per_step": int(h2d), "d2h_bytes_per_step": int(d2h),
                       "what": "spsyrk_host_tril: H2D of A, plan+symbolic+numeric, D2H of C_L (mirror not included)"}

    if rank == 0 and world == 1 and not args.skip_extras and not args.no_cpu:
        s = oracle_sample(a, 1, 0)
        line["cpu_baseline"] = {"value": s["macs"] / s["times"][0], "unit": UNIT, "cores": 1, "kind": "oracle",
                                "sample": f"rows [{s['r0']}, {s['r0'] + s['rows']}) of {a.name}: {s['macs']} multiply-adds in {s['times'][0]:.2f} s"}
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
