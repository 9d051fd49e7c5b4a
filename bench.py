#!/usr/bin/env python
"""Benchmark of the fused star-join query pipeline.

    python bench.py --gpus N --steps K --warmup W            (one rank per GPU under torchrun for N > 1)
    python bench.py --impl reference --gpus N --steps K --warmup W

A step is one whole query: plan and build every dimension table from the
filtered dimension columns, then one fused pass over the fact table (and, for
N > 1, an all-reduce of the dense result).  The workload is the four-join
group-by over 600 M fact rows (14.4 GB of referenced fact columns, far larger
than the 126 MB L2, so no L2 flush is needed between steps); every rank holds
its own 600 M-row shard of the row space and a replica of the dimensions
(weak scaling).  Rank 0 prints ONE JSON line.
"""
from __future__ import annotations

import argparse
import json
import os
import sys
import threading
import time

ROOT = os.path.dirname(os.path.abspath(__file__))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

METRIC = "fact_rows_per_s"
UNIT = "rows/s"
CONTRACT_HBM_GBS = 8000.0
FALLBACK_HBM_GBS = 6650.0
# DRAM bytes per fact row of the fused kernel, from an ncu capture of a 100 M-row case of the same workload
# (dram__bytes_read.sum + dram__bytes_write.sum; traffic grows in proportion to the rows)
NCU_DRAM_BYTES_PER_ROW = {"c3": 12.2}


def measured_hbm_peak():
    try:
        with open(os.path.join(ROOT, "MEASURED_PEAKS.json")) as f:
            return float(json.load(f)["hbm_gbs"]), "measured"
    except Exception:
        return FALLBACK_HBM_GBS, "fallback"


def make_workload(name: str, rows: int | None, sel: float, groups: int):
    from datagen import workloads as W

    if name == "c4":
        return W.config4(rows or 600_000_000, sel, groups)
    return W.CONFIGS[name](rows) if rows else W.CONFIGS[name]()


def stage_selectivities(w):
    """Exact pass fractions of the workload's filters, from its definition (uniform draws)."""
    from datagen import DATE_ROWS

    sel = {}
    if w.name.startswith("c1"):
        sel = {"pred:discount": 3 / 11, "pred:quantity": 29 / 50, "join:date": 365 / DATE_ROWS}
    elif w.name.startswith("c2"):
        sel = {"join:part": 1 / 25, "join:supplier": 1 / 5, "join:date": 1.0}
    elif w.name.startswith("c3"):
        sel = {"join:customer": 1 / 5, "join:supplier": 1 / 5, "join:part": 2 / 5, "join:date": 729 / DATE_ROWS}
    elif w.name.startswith("c4"):
        sel = {"pred:p": w.preds[0].lo / 10000.0, "join:dim": 1.0}
    elif w.name.startswith("c5"):
        sel = {"join:dim": 0.25}
    return sel


def algorithmic_bytes_per_row(w, order):
    """Sector model: the first column is read whole; a later column is read for a 32-byte sector
    iff at least one of its rows survived everything evaluated before it."""
    sel = stage_selectivities(w)
    names = [f"pred:{p.col}" for p in w.preds] + [f"join:{d}" for _, d in w.joins]
    cols = [p.col for p in w.preds] + [fk for fk, _ in w.joins]
    reach, total, seen, applied = 1.0, 0.0, set(), set()
    for idx in order:
        if idx < 0 or idx in applied:  # a repeated label is the gather copy of a filter stage: nothing new is read
            continue
        applied.add(idx)
        col = cols[idx]
        width = 8 if w.fact_col(col).is64 else 4
        if col not in seen:
            total += width * (1.0 - (1.0 - reach) ** (32 // width))
            seen.add(col)
        reach *= sel.get(names[idx], 1.0)
    for c in w.fact_cols:  # columns only the key or the aggregate reads
        if c.name not in seen:
            width = 8 if c.is64 else 4
            total += width * (1.0 - (1.0 - reach) ** (32 // width))
    return total


class ClockSampler(threading.Thread):
    """Samples SM clock and throttle reasons of one GPU through NVML while the timed region runs.  NVML is
    initialised before the thread starts, so that a short timed region is covered from its first milliseconds
    (an NVML query takes milliseconds: it must not sit in the timing loop itself)."""

    def __init__(self, index: int):
        super().__init__(daemon=True)
        self.index, self.stop_flag, self.samples, self.reasons, self.max_mhz = index, False, [], set(), None
        self.error = None
        self.nv = self.handle = None
        self.names = {}
        try:
            import pynvml as nv

            nv.nvmlInit()
            self.nv = nv
            self.handle = nv.nvmlDeviceGetHandleByIndex(self.index)
            self.max_mhz = nv.nvmlDeviceGetMaxClockInfo(self.handle, nv.NVML_CLOCK_SM)
            self.names = {nv.nvmlClocksEventReasonHwSlowdown: "hw_slowdown",
                          nv.nvmlClocksEventReasonHwThermalSlowdown: "hw_thermal_slowdown",
                          nv.nvmlClocksEventReasonSwThermalSlowdown: "sw_thermal_slowdown",
                          nv.nvmlClocksEventReasonSwPowerCap: "sw_power_cap"}
        except Exception as e:  # pragma: no cover - depends on the box
            self.error = repr(e)

    def sample(self):
        if self.handle is None:
            return
        try:
            nv = self.nv
            self.samples.append(nv.nvmlDeviceGetClockInfo(self.handle, nv.NVML_CLOCK_SM))
            try:
                r = nv.nvmlDeviceGetCurrentClocksEventReasons(self.handle)
            except Exception:
                r = nv.nvmlDeviceGetCurrentClocksThrottleReasons(self.handle)
            for bit, nm in self.names.items():
                if r & bit:
                    self.reasons.add(nm)
        except Exception as e:  # pragma: no cover
            self.error = repr(e)

    def run(self):
        while not self.stop_flag:
            self.sample()
            time.sleep(0.01)

    def summary(self):
        if not self.samples:
            return {"sm_mhz": None, "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons), "samples": 0,
                    "error": self.error}
        s = sorted(self.samples)
        return {"sm_mhz": s[len(s) // 2], "sm_max_mhz": self.max_mhz, "reasons": sorted(self.reasons),
                "samples": len(s)}


def visible_gpu_index(local_rank: int) -> int:
    vis = os.environ.get("CUDA_VISIBLE_DEVICES")
    if vis:
        try:
            return int(vis.split(",")[local_rank])
        except Exception:
            return local_rank
    return local_rank


def oracle_rate(w, sample_rows: int, row0: int = 0):
    """Time the CPU oracle (as it stands, one thread) on rows [row0, row0 + sample_rows) of the workload."""
    import oracle
    from datagen import workloads as W

    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    fact = W.host_fact(w, row0, sample_rows)
    t0 = time.perf_counter()
    dims = oracle.build_dims(w, hd)
    t_build = time.perf_counter() - t0
    r = oracle.run(w, fact, dims)
    return sample_rows / (r["seconds"] + t_build), r["seconds"], t_build


def run_reference(args):
    """The reference arm: the CPU oracle, as it stands, on bounded samples of the same workload."""
    rank = int(os.environ.get("RANK", "0"))
    if rank != 0:
        return 0
    import oracle
    from datagen import workloads as W

    w = make_workload(args.workload, args.rows, args.sel, args.groups)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    probe = min(w.n_rows, 2_000_000)
    fact = W.host_fact(w, 0, probe)
    dims = oracle.build_dims(w, hd)
    t = oracle.run(w, fact, dims)["seconds"]
    per_row = max(t / probe, 1e-9)
    wall_s = 90.0  # total CPU time the reference arm may take
    sample = int(min(w.n_rows, max(100_000, wall_s / per_row / (args.steps + args.warmup))))
    times = []
    for i in range(args.warmup + args.steps):
        row0 = (i * sample) % max(1, w.n_rows - sample + 1)
        fact = W.host_fact(w, row0, sample)
        t0 = time.perf_counter()
        dims = oracle.build_dims(w, hd)
        oracle.run(w, fact, dims)
        dt = time.perf_counter() - t0
        if i >= args.warmup:
            times.append(dt)
    ms = 1000.0 * sum(times) / len(times)
    value = sample / (ms / 1000.0)
    line = {"impl": "reference", "metric": METRIC, "value": value, "unit": UNIT, "n_gpus": args.gpus,
            "steps": args.steps, "warmup": args.warmup, "ms_per_step": ms, "higher_is_better": True,
            "scaling": "weak", "vs_baseline": None, "dtype": "int64", "data": "synthetic",
            "config": {"workload": w.name, "rows": w.n_rows, "rows_per_step": sample,
                       "note": "CPU oracle (single thread) on a bounded sample of the workload per step"},
            "cpu_baseline": {"value": value, "unit": UNIT, "cores": 1, "kind": "oracle",
                             "sample": f"{sample} consecutive fact rows per step, dimension build included"},
            "e2e": {"value": value, "unit": UNIT, "h2d_bytes_per_step": 0, "d2h_bytes_per_step": 0},
            "gpu_launches": 0}
    print(json.dumps(line), flush=True)
    return 0


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4", "c5"])
    ap.add_argument("--rows", type=int, default=None, help="override the fact rows per GPU (debugging)")
    ap.add_argument("--sel", type=float, default=0.1, help="c4: fact predicate selectivity")
    ap.add_argument("--groups", type=int, default=1000, help="c4: number of groups")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--cpu-sample-rows", type=int, default=100_000_000)
    ap.add_argument("--interpret", action="store_true",
                    help="interpret the query descriptor instead of compiling the fused kernel for the query's shape")
    ap.add_argument("--block-threads", type=int, default=0,
                    help="force the fused kernel's block size (profiling a small case in the full-size launch shape)")
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--extras", action="store_true", help="also time the other configurations (N = 1 only)")
    ap.add_argument("--ablation", action="store_true",
                    help="also run the A/B switches (lazy vs eager loads, queues, table forms, group-by paths)")
    args = ap.parse_args()
    if args.warmup < 3:
        args.warmup = 3
    if args.impl == "reference":
        return run_reference(args)

    import torch
    import torch.distributed as dist

    from paper_2607_07632_b200 import build as sjq_build

    if int(os.environ.get("LOCAL_RANK", "0")) == 0:
        sjq_build.build()  # compiles libsjq.so only if it is missing or older than its sources
    import paper_2607_07632_b200 as sjq
    from datagen import workloads as W
    from paper_2607_07632_b200 import shard

    rank = int(os.environ.get("RANK", "0"))
    local_rank = int(os.environ.get("LOCAL_RANK", "0"))
    world = int(os.environ.get("WORLD_SIZE", "1"))
    if not torch.cuda.is_available():
        raise SystemExit("bench.py needs a CUDA device: the product path has no CPU fallback")
    torch.cuda.set_device(local_rank)
    device = torch.device("cuda", local_rank)
    if world > 1:
        os.environ.setdefault("MASTER_ADDR", "127.0.0.1")
        dist.init_process_group("nccl", device_id=device)

    w = make_workload(args.workload, args.rows, args.sel, args.groups)
    n = w.n_rows
    dims = {d.name: W.device_dim(w, d, device) for d in w.dims}
    fact = W.device_fact(w, row0=rank * n, n=n, device=device)  # this rank's shard of the row space
    torch.cuda.synchronize()

    # every event pair is created (recorded once) up front; the library records them around the fused kernel
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range(args.steps)]
    for a, b in pairs:
        a.record()
        b.record()
    res = sjq.alloc_result(w.mode, w.num_groups, w.capacity, w.agg.want_count, device)
    builders = sjq.workload_builders(w, dims)  # argument marshalling done once; plan + build run every step
    launches = 0
    info = None

    def step(i=None):
        nonlocal launches, info
        tables = sjq.build_tables(builders)
        opts = sjq.RunOpts(events=pairs[i] if i is not None else None, specialise=not args.interpret,
                           block_threads=args.block_threads, ctas_per_sm=args.ctas_per_sm)
        r = sjq.run_workload(w, fact, tables, opts, result=res)
        if world > 1 and w.mode != "HASHED":
            shard.merge_dense(res.sums, res.counts)
        if i is not None:
            launches += r.info.kernel_launches + sum(sjq.build_launches(t) for t in tables.values())
        info = r.info
        return tables

    if not args.interpret:
        # the first specialised run compiles the kernel; if the compiler is not available on this machine say so
        # and time the interpreted kernel (still the library's CUDA path) rather than nothing
        try:
            step()
        except sjq.SjqError as ex:
            if ex.status != 7:
                raise
            print(f"bench.py: run-time specialisation unavailable ({ex}); {sjq.jit_log()[:300]!r}; "
                  "timing the interpreted kernel", file=sys.stderr, flush=True)
            args.interpret = True
    for _ in range(args.warmup):
        tables = step()
    torch.cuda.synchronize()
    assert res.status() == 0 and all(t.status() == 0 for t in tables.values())

    sampler = ClockSampler(visible_gpu_index(local_rank))
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev0.record()
    for i in range(args.steps):
        step(i)
    ev1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.stop_flag = True
    sampler.join(timeout=2.0)
    ms_total = ev0.elapsed_time(ev1)
    fused_ms = sum(a.elapsed_time(b) for a, b in pairs) / len(pairs)
    t = torch.tensor([ms_total, fused_ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total, fused_ms = float(t[0]), float(t[1])
    ms_per_step = ms_total / args.steps
    value = world * n / (ms_per_step / 1000.0)
    ref_bytes = w.referenced_bytes_per_row()
    eff_gbs = world * n * ref_bytes / (ms_per_step / 1000.0) / 1e9

    peak, peak_kind = measured_hbm_peak()
    alg_bpr = algorithmic_bytes_per_row(w, list(info.order[: info.nstages]))
    achieved = n * alg_bpr / (fused_ms / 1000.0) / 1e9
    traffic_bpr = NCU_DRAM_BYTES_PER_ROW.get(args.workload)
    roofline = {"bound": "hbm", "kernel": "fused_kernel" if args.interpret else "sjq_jit_kernel", "achieved": achieved, "peak": peak,
                "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic_bpr * n if traffic_bpr else None,
                "algorithmic_bytes_per_row": alg_bpr, "kernel_ms": fused_ms,
                "effective_gbs_kernel": n * ref_bytes / (fused_ms / 1000.0) / 1e9}

    e2e = None
    if not args.no_e2e:
        try:
            host_fact = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in fact.items()}
            for k, v in fact.items():
                host_fact[k].copy_(v)
            torch.cuda.synchronize()
            chunk = min(n, 32 << 20) // 4 * 4 or 4
            staging = torch.empty(sjq.staging_bytes(host_fact, chunk), dtype=torch.uint8, device=device)
            eres, ehost = None, None

            def e2e_step():
                nonlocal eres, ehost
                tabs = sjq.build_tables(builders)
                eres, ehost = sjq.run_workload_host(w, host_fact, tabs, staging, chunk,
                                                    sjq.RunOpts(specialise=not args.interpret), result=eres, host=ehost)
                torch.cuda.synchronize()  # the result is on the host when this returns
                return tabs

            tabs = e2e_step()
            if world > 1:
                dist.barrier()
            t0 = time.perf_counter()
            for _ in range(args.e2e_steps):
                e2e_step()
            dt = (time.perf_counter() - t0) / args.e2e_steps
            tt = torch.tensor([dt], dtype=torch.float64, device=device)
            if world > 1:
                dist.all_reduce(tt, op=dist.ReduceOp.MAX)
            dt = float(tt[0])
            same = bool(torch.equal(ehost.sums, res.sums.cpu())) if world == 1 else None
            cells = 1 if w.mode == "SCALAR" else w.num_groups if w.mode == "DENSE" else w.capacity
            # bytes over the bus: whole columns for the copied ones; for a column the kernel reads in place, the
            # 32-byte sectors holding a surviving row (estimated from the planner's share of rows reaching it)
            plan = sjq.host_transfer_plan({c.name: host_fact[c.name] for c in w.fact_cols}, w.preds,
                                          [(fk, tabs[dn]) for fk, dn in w.joins], w.key, w.agg,
                                          sjq.RunOpts(specialise=not args.interpret))
            copied = sum(n * host_fact[k].element_size() for k, (how, _) in plan.items() if how == "copy")
            in_place = sum(n * host_fact[k].element_size() * (1.0 - (1.0 - sh) ** (32 // host_fact[k].element_size()))
                           for k, (how, sh) in plan.items() if how == "in place")
            e2e = {"value": world * n / dt, "unit": UNIT, "h2d_bytes_per_step": int(copied + in_place),
                   "h2d_copied_bytes": int(copied), "h2d_in_place_bytes_estimate": int(in_place),
                   "columns": {k: how for k, (how, _) in plan.items()},
                   "d2h_bytes_per_step": cells * 8 * (2 if w.agg.want_count else 1) + 4, "ms_per_step": dt * 1000.0,
                   "steps": args.e2e_steps, "chunk_rows": chunk, "matches_device_run": same,
                   "api": "sjq_run_host (pinned host columns: chunked double-buffered copies of the columns most rows need, "
                          "in-place reads of the sparse ones, result copied back)"}
            del host_fact, staging
        except Exception as ex:  # e.g. not enough page-locked memory on the box
            e2e = {"value": None, "unit": UNIT, "error": repr(ex)[:200]}

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = min(n, args.cpu_sample_rows)
        rate, secs, tb = oracle_rate(w, sample)
        cpu = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {sample} fact rows of the workload; row loop {secs:.2f} s + dimension maps {tb:.2f} s",
               "host_cores_available": os.cpu_count()}

    extras = None
    if args.extras and world == 1 and rank == 0:
        del fact
        torch.cuda.empty_cache()
        extras = run_extras(sjq, W, device, not args.interpret)
    ablation = None
    if args.ablation and world == 1 and rank == 0:
        if "fact" in locals():
            del fact
        torch.cuda.empty_cache()
        ablation = run_ablation(sjq, W, device, not args.interpret)

    if rank == 0:
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": "weak",
                "vs_baseline": None, "dtype": "int64", "data": "synthetic",
                "config": {"workload": w.name, "rows_per_gpu": n, "referenced_bytes_per_row": ref_bytes,
                           "step": "plan+build of every dimension table (on side streams; the key-range scans may overlap the previous step's fused pass), then the fused pass"
                                   + (", then all-reduce of the dense result" if world > 1 else ""),
                           "l2": "inputs (%.1f GB) exceed the 126 MB L2; no flush needed" % (n * ref_bytes / 1e9),
                           "parallelism": f"row-sharded x{world}, dimensions replicated", "plan": info.describe(),
                           "fused_kernel": "interpreted descriptor" if args.interpret else
                                           "compiled for the query's shape at run time during warm-up (NVRTC), cached"},
                "effective_gbs": eff_gbs, "pct_of_8tbs": 100.0 * eff_gbs / world / CONTRACT_HBM_GBS,
                "pct_of_measured_copy_peak": 100.0 * eff_gbs / world / peak,
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches,
                "clocks": sampler.summary()}
        if extras is not None:
            line["other_configs"] = extras
        if ablation is not None:
            line["ablation"] = ablation
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def run_extras(sjq, W, device, specialise=True):
    """Run-only timings (tables prebuilt) of the other configurations: min and mean of 10 after a warm-up."""
    import torch

    out = []

    def timed(w):
        dims = {d.name: W.device_dim(w, d, device) for d in w.dims}
        tables = sjq.build_workload_tables(w, dims)
        fact = W.device_fact(w, device=device)
        opts = sjq.RunOpts(specialise=specialise)
        res = sjq.run_workload(w, fact, tables, opts)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ts = []
        for _ in range(10):
            e0.record()
            sjq.run_workload(w, fact, tables, opts, result=res)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        eff = w.n_rows * w.referenced_bytes_per_row() / (min(ts) / 1000.0) / 1e9
        out.append({"workload": w.name, "rows": w.n_rows, "ms_min": min(ts), "ms_mean": sum(ts) / len(ts),
                    "rows_per_s": w.n_rows / (min(ts) / 1000.0), "effective_gbs": eff,
                    "pct_of_8tbs": 100.0 * eff / CONTRACT_HBM_GBS, "status": res.status(),
                    "plan": res.info.describe()})
        del fact, tables, dims, res
        torch.cuda.empty_cache()

    timed(W.config1())
    timed(W.config2())
    timed(W.config5())
    timed(W.city_pair())  # beyond the five configurations: many groups, few survivors
    for s in (0.0001, 0.01, 0.1, 0.5, 1.0):
        for g in (1, 1000, 100000, 1000000):
            timed(W.config4(600_000_000, s, g))
    # the large group counts as DENSE results too (global atomics, no key look-up), for comparison with the
    # hashed form the configuration asks for
    for s in (0.1, 1.0):
        for g in (100000, 1000000):
            timed(W.config4(600_000_000, s, g, hashed=False))
    return out


def run_ablation(sjq, W, device, specialise=True):
    """The paper's A/B experiments restated on this kernel (run-only, min of 5 after a warm-up):
    lazy vs unconditional column loads (its tile-vs-direct table), survivor queues on/off, packed
    direct-mapped vs open-addressing tables, privatised vs global group-by (its ablation figure)."""
    import torch

    out = []

    def timed(w, label, opts=None, force_hash=False, tables=None, fact=None, dims=None):
        if dims is None:
            dims = {d.name: W.device_dim(w, d, device) for d in w.dims}
        if tables is None:
            tables = {d.name: sjq.build_dim(dims[d.name], d.key, d.preds, d.payloads,
                                            force_kind=sjq.sjq.FORCE_HASH if (force_hash or d.force_hash) else 0)
                      for d in w.dims}
        if fact is None:
            fact = W.device_fact(w, device=device)
        if opts is None:
            opts = sjq.RunOpts()
        if label != INTERPRETED:
            opts.specialise = specialise
        res = sjq.run_workload(w, fact, tables, opts)
        torch.cuda.synchronize()
        e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
        ts = []
        for _ in range(5):
            e0.record()
            sjq.run_workload(w, fact, tables, opts, result=res)
            e1.record()
            torch.cuda.synchronize()
            ts.append(e0.elapsed_time(e1))
        out.append({"workload": w.name, "variant": label, "ms_min": min(ts),
                    "rows_per_s": w.n_rows / (min(ts) / 1000.0), "status": res.status(),
                    "table_kinds": {k: t.layout.kind_name for k, t in tables.items()},
                    "table_bytes": {k: int(t.layout.table_bytes) for k, t in tables.items()},
                    "plan": res.info.describe()})
        return fact, dims

    INTERPRETED = "query descriptor interpreted (no run-time specialisation)"
    for mk in (W.config3, W.config2):
        w = mk()
        fact, dims = timed(w, "default")
        for label, opts in ((INTERPRETED, sjq.RunOpts()),
                            ("eager loads (every column for every row)", sjq.RunOpts(eager_loads=True)),
                            ("no survivor queues (thread-owned rows throughout)", sjq.RunOpts(compaction=1)),
                            ("one queue only", sjq.RunOpts(compaction=2)),
                            ("global atomics group-by", sjq.RunOpts(agg_path=2)),
                            ("shared-memory privatised group-by", sjq.RunOpts(agg_path=1)),
                            ("every direct table in shared memory that fits", sjq.RunOpts(smem_tables=2)),
                            ("no table in shared memory", sjq.RunOpts(smem_tables=1)),
                            ("filter stages probe the packed code arrays, not their presence bitmaps",
                             sjq.RunOpts(no_filter_bitmap=True))):
            try:
                timed(w, label, opts, fact=fact, dims=dims)
            except sjq.SjqError as e:
                out.append({"workload": w.name, "variant": label, "error": str(e)})
        timed(w, "open-addressing tables instead of packed direct maps", None, force_hash=True, fact=fact, dims=dims)
        del fact, dims
        torch.cuda.empty_cache()
    # hashed result over a million groups: the table indexed by the key (what a modulo key allows) vs the hash table
    w = W.config4(600_000_000, 0.1, 1000000)
    fact, dims = timed(w, "default")
    timed(w, "group hash table instead of the direct-indexed group table", sjq.RunOpts(group_hash_always=True),
          fact=fact, dims=dims)
    del fact, dims
    torch.cuda.empty_cache()
    return out


if __name__ == "__main__":
    sys.exit(main())
