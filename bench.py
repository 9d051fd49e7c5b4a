#!/usr/bin/env python
"""Benchmark of the fused star-join query pipeline.

    python bench.py --gpus N --steps K --warmup W            (one rank per GPU under torchrun for N > 1)
    python bench.py --impl reference --gpus N --steps K --warmup W

A step is one whole query: plan and build every dimension table from the
filtered dimension columns, then one fused pass over the fact table (and, for
N > 1, the merge of the per-rank results: one all-reduce, or for a hashed
result one all-gather and a merge kernel).  The workload is the four-join
group-by over 600 M fact rows (14.4 GB of referenced fact columns, far larger
than the 126 MB L2, so no L2 flush is needed between steps); every rank holds
its own 600 M-row shard of the row space and a replica of the dimensions
(weak scaling; `--scaling strong` cuts one 1.2 B-row table over the ranks
instead).  Rank 0 prints ONE JSON line.  At N = 1 the line also carries
`points`: every other configuration (config 1, 2, 5, the 20 points of the
selectivity x cardinality sweep, the two high-cardinality shapes), each run
ten times or more with its own roofline figures, clock record and a bit-exact
comparison with the oracle-written expected values under tests/golden/.
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
# (dram__bytes_read.sum + dram__bytes_write.sum; traffic grows in proportion to the rows), each with the plan
# it was captured under: the figure is reported only while the running plan is that one.
NCU_PROFILED = {
    "c3_four_join_groupby": {"dram_bytes_per_row": 12.2, "kernel": "sjq_jit_kernel",
                             "order": [1, 3, 0, 2, 3, 0, -1, -1], "block": 1024, "queue_levels": 3,
                             "summary": "profiles/fused_kernel_c3_100m.md"},
}


def profiled_traffic(w, info, kernel, rows):
    """(bytes per launch, note): the ncu DRAM traffic scaled to `rows`, or None when the plan that ran is not
    the plan the capture was taken under."""
    p = NCU_PROFILED.get(w.name)
    if p is None:
        return None, "no capture of this workload"
    plan = info.describe()
    same = (plan["order"] == p["order"] and plan["block"] == p["block"] and plan["queue_levels"] == p["queue_levels"]
            and kernel == p["kernel"])
    if not same:
        return None, f"the plan that ran differs from the one captured in {p['summary']}"
    return p["dram_bytes_per_row"] * rows, p["summary"]


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
    mk = W.CONFIGS.get(name) or W.EXTRA_SHAPES[name]
    return mk(rows) if rows else mk()


def _uniform_pred_fraction(c, p):
    """Exact share of U[a, b] that passes predicate p (None when the column is not a plain uniform draw)."""
    from datagen import UNIFORM_I32

    if c.kind != UNIFORM_I32:
        return None
    a, b = c.a, c.b
    n = b - a + 1

    def below(x):  # values of [a, b] that are < x
        return min(max(x - a, 0), n)

    if p.op == "EQ":
        k = 1 if a <= p.lo <= b else 0
    elif p.op == "NE":
        k = n - (1 if a <= p.lo <= b else 0)
    elif p.op == "LT":
        k = below(p.lo)
    elif p.op == "LE":
        k = below(p.lo + 1)
    elif p.op == "GT":
        k = n - below(p.lo + 1)
    elif p.op == "GE":
        k = n - below(p.lo)
    elif p.op == "BETWEEN":
        k = max(0, min(b, p.hi) - max(a, p.lo) + 1)
    else:
        k = len({v for v in p.values if a <= v <= b})
    return k / n


def stage_pass_fractions(w, tables, survivors=None):
    """Pass fraction of every filter of the workload, label -> fraction, labels as in the plan's `order`
    (predicate index, then number of predicates + join index).  Predicates on uniform columns and joins whose
    foreign key is drawn uniformly over the dimension's rows are exact by construction (rows passing the
    dimension filter / rows of the dimension, as the built table reports them); one remaining unknown (the
    Zipf-distributed key of config 5) is solved from the survivor count of the run."""
    from datagen import DATE_FK_I32, SEQ_I32, DATE_KEY_I32, UNIFORM_I32

    frac = {}
    for i, p in enumerate(w.preds):
        frac[i] = _uniform_pred_fraction(w.fact_col(p.col), p)
    for j, (fk, dn) in enumerate(w.joins):
        c, d, L = w.fact_col(fk), w.dim(dn), tables[dn].layout
        key_kind = next(x.kind for x in d.cols if x.name == d.key)
        uniform = (c.kind == UNIFORM_I32 and key_kind == SEQ_I32 and c.a == 1 and c.b == d.rows) or \
                  (c.kind == DATE_FK_I32 and key_kind == DATE_KEY_I32)
        frac[len(w.preds) + j] = (L.entries / L.dim_rows) if (uniform and L.dim_rows) else None
    unknown = [k for k, v in frac.items() if v is None]
    if len(unknown) == 1 and survivors is not None and w.n_rows:
        known = 1.0
        for v in frac.values():
            known *= v if v is not None else 1.0
        frac[unknown[0]] = min(1.0, survivors / w.n_rows / known) if known > 0 else 1.0
    return {k: (1.0 if v is None else v) for k, v in frac.items()}


def algorithmic_bytes_per_row(w, order, frac, granule: int = 32):
    """Sector model: the first column is read whole; a later column is read for a 32-byte sector
    iff at least one of its rows survived everything evaluated before it.  `order`: the stage labels of
    the plan that ran; `frac`: pass fraction per label.  granule = 64 gives the same model for 64-byte
    pieces, the smallest unit DRAM delivered in the ncu captures (reported beside the 32-byte figure,
    never instead of it)."""
    cols = [p.col for p in w.preds] + [fk for fk, _ in w.joins]
    reach, total, seen, applied = 1.0, 0.0, set(), set()
    for idx in order:
        if idx < 0 or idx in applied:  # a repeated label is the gather copy of a filter stage: nothing new is read
            continue
        applied.add(idx)
        col = cols[idx]
        width = 8 if w.fact_col(col).is64 else 4
        if col not in seen:
            total += width * (1.0 - (1.0 - reach) ** (granule // width))
            seen.add(col)
        reach *= frac.get(idx, 1.0)
    referenced = set(cols) | {t.a for t in ((w.key.terms if w.key and w.key.modulo != 1 else ()) + (w.agg.x,) +
                                            ((w.agg.y,) if w.agg.y is not None else ())) if t.src == "FACT"}
    for c in w.fact_cols:  # columns only the key or the aggregate reads
        if c.name not in seen and c.name in referenced:
            width = 8 if c.is64 else 4
            total += width * (1.0 - (1.0 - reach) ** (granule // width))
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


def golden_for(w):
    """Expected result written by the CPU oracle for this workload at this size (tests/golden/full_*.json), or None."""
    from datagen import workloads as W

    if w.name.startswith("c4_sweep"):
        sel = next(s for s, t in W.C4_THRESHOLDS.items() if t == w.preds[0].lo)
        tag = f"c4_s{sel:g}_g{w.key.modulo}"
    else:
        tag = {"c1_filter_agg": "c1", "c2_two_join_groupby": "c2", "c3_four_join_groupby": "c3",
               "c5_skewed_sparse": "c5", "city_pair_groupby": "city_pair", "city_brand_groupby": "city_brand",
               "city_brand_groupby_dense": "city_brand"}.get(w.name)
    path = os.path.join(ROOT, "tests", "golden", f"full_{tag}.json")
    if tag is None or not os.path.exists(path):
        return None
    with open(path) as f:
        g = json.load(f)
    return g if g["rows"] == w.n_rows else None


def matches_golden(w, res, g):
    """True iff the device result equals the stored expected values bit for bit (None: nothing stored)."""
    import hashlib

    import numpy as np

    if g is None:
        return None
    if w.mode == "SCALAR":
        return int(res.sums[0].item()) == g["sum"] and int(res.counts[0].item()) == g["count"]

    def digest(*arrays):
        h = hashlib.sha256()
        for a in arrays:
            h.update(np.ascontiguousarray(a, dtype="<i8").tobytes())
        return h.hexdigest()

    if w.mode == "DENSE":
        s, c = res.sums.cpu().numpy(), res.counts.cpu().numpy()
        if "sums" in g:
            return s.tolist() == g["sums"] and c.tolist() == g["counts"]
        if g.get("mode") == "HASHED":  # stored as a list: compare the non-empty groups of the dense array
            keys = np.nonzero(c)[0]
            return keys.size == g["groups"] and digest(keys, s[keys], c[keys]) == g["sha256"]
        return digest(s, c) == g["dense_sha256"]
    k, s, c = (t.cpu().numpy() for t in res.hashed_sorted())
    if "sha256" in g:
        return k.size == g["groups"] and digest(k, s, c) == g["sha256"]
    # stored as a dense array: scatter the list
    full_s, full_c = np.zeros(w.num_groups, np.int64), np.zeros(w.num_groups, np.int64)
    full_s[k], full_c[k] = s, c
    return digest(full_s, full_c) == g["dense_sha256"]


def measure_point(sjq, torch, w, fact, tables, specialise, gpu_index, peak, extra_opts=None, min_runs=10,
                  min_busy_ms=60.0):
    """Run-only measurement of one workload (tables prebuilt): at least `min_runs` calls of sjq_run enqueued
    back to back (more, until the GPU has been busy for `min_busy_ms`, so that the clock sampler sees the
    point under load), each timed with its own CUDA events: the whole call (clear + fused kernel + compaction)
    and the fused kernel alone."""
    kw = dict(extra_opts or {})
    # planning: the fact predicates' pass fractions are measured once (outside the timed runs, like the table builds)
    kw["pass_ppm"] = sjq.sample_preds({c.name: fact[c.name] for c in w.fact_cols}, w.preds)
    res = sjq.run_workload(w, fact, tables, sjq.RunOpts(specialise=specialise, **kw))
    torch.cuda.synchronize()
    e0, e1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    e0.record()
    sjq.run_workload(w, fact, tables, sjq.RunOpts(specialise=specialise, **kw), result=res)
    e1.record()
    torch.cuda.synchronize()
    runs = int(min(200, max(min_runs, min_busy_ms / max(e0.elapsed_time(e1), 1e-3))))
    ref_bytes = w.referenced_bytes_per_row()
    small = w.n_rows * ref_bytes < (512 << 20)  # may sit in the 126 MB L2: evict it between runs
    flush = torch.empty(256 << 20, dtype=torch.uint8, device=res.sums.device) if small else None
    outer = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(runs)]
    inner = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)) for _ in range(runs)]
    for a, b in inner:
        a.record()
        b.record()
    sampler = ClockSampler(gpu_index)
    torch.cuda.synchronize()
    sampler.sample()
    sampler.start()
    for i in range(runs):
        if flush is not None:
            flush.zero_()
        outer[i][0].record()
        sjq.run_workload(w, fact, tables, sjq.RunOpts(specialise=specialise, events=inner[i], **kw), result=res)
        outer[i][1].record()
    torch.cuda.synchronize()
    sampler.sample()
    sampler.stop_flag = True
    sampler.join(timeout=2.0)
    ms = [a.elapsed_time(b) for a, b in outer]
    kms = [a.elapsed_time(b) for a, b in inner]
    status = res.status()
    info = res.info
    if w.mode == "HASHED":
        survivors = int(res.counts[: int(res.n_groups.item())].sum().item())
    else:
        survivors = int(res.counts.sum().item()) if res.counts is not None else None
    frac = stage_pass_fractions(w, tables, survivors)
    plan = info.describe()
    alg = algorithmic_bytes_per_row(w, plan["order"], frac)
    ms_mean, k_mean = sum(ms) / runs, sum(kms) / runs
    achieved = w.n_rows * alg / (k_mean / 1000.0) / 1e9
    eff = w.n_rows * ref_bytes / (k_mean / 1000.0) / 1e9
    out = {"workload": w.name, "rows": w.n_rows, "runs": runs, "ms_min": min(ms), "ms_mean": ms_mean,
           "kernel_ms_min": min(kms), "kernel_ms_mean": k_mean, "rows_per_s": w.n_rows / (ms_mean / 1000.0),
           "algorithmic_bytes_per_row": alg, "achieved_gbs": achieved, "frac": achieved / peak,
           "bytes_per_row_64B_model": algorithmic_bytes_per_row(w, plan["order"], frac, 64),
           "referenced_bytes_per_row": ref_bytes, "effective_gbs_kernel": eff,
           "pct_of_8tbs": 100.0 * eff / CONTRACT_HBM_GBS, "survivors": survivors,
           "pass_fractions": {str(k): round(v, 6) for k, v in frac.items()},
           "sampled_pass_ppm": list(kw["pass_ppm"]),
           "l2": "256 MB written between runs" if small else "inputs exceed the L2",
           "status": status, "parity": matches_golden(w, res, golden_for(w)) if status == 0 else False,
           "plan": plan, "table_kinds": {k: t.layout.kind_name for k, t in tables.items()},
           "clocks": sampler.summary()}
    if plan["agg_path"] in ("global", "hash") and survivors is not None:
        # one 64-bit atomic add per survivor for the sum and one for the count where counts are kept
        per_row = 2 if (w.agg.want_count or w.mode == "HASHED") else 1
        out["atomic_adds_per_s"] = survivors * per_row / (k_mean / 1000.0)
    return out


def run_points(sjq, torch, W, device, specialise, gpu_index, peak, c3_inputs=None, extras=False):
    """Every configuration besides the headline one, run-only, each with its own figures and parity."""
    out = []

    def inputs(w):
        dims = {d.name: W.device_dim(w, d, device) for d in w.dims}
        return W.device_fact(w, device=device), sjq.build_workload_tables(w, dims)

    def point(w, fact=None, tables=None, **kw):
        if fact is None:
            fact, tables = inputs(w)
        try:
            out.append(measure_point(sjq, torch, w, fact, tables, specialise, gpu_index, peak, **kw))
        except Exception as ex:  # one failing point must not hide the others
            out.append({"workload": w.name, "rows": w.n_rows, "error": repr(ex)[:300], "parity": False})
        return fact, tables

    if c3_inputs is not None:
        point(*c3_inputs)
        c3_inputs[1].clear()  # the caller's columns are not needed any more: free them
        torch.cuda.empty_cache()
    for mk in (W.config1, W.config2, W.config5, W.city_pair, W.city_brand):
        point(mk())
        torch.cuda.empty_cache()
    if extras:
        point(W.city_brand(hashed=False))  # the same query asked for as the dense array of all 1.75 M groups
        torch.cuda.empty_cache()
    # the sweep: its four fact columns and its dimension do not depend on the threshold or the group count
    fact = tables = None
    for s in W.C4_THRESHOLDS:
        for g in W.C4_GROUPS:
            fact, tables = point(W.config4(600_000_000, s, g), fact, tables)
    if extras:
        # the large group counts as DENSE results too (no key list), and through the group hash table
        for s in (0.1, 1.0):
            for g in (100000, 1000000):
                point(W.config4(600_000_000, s, g, hashed=False), fact, tables)
                point(W.config4(600_000_000, s, g), fact, tables, extra_opts={"group_hash_always": True})
    del fact, tables
    torch.cuda.empty_cache()
    return out


def main():
    ap = argparse.ArgumentParser()
    ap.add_argument("--gpus", type=int, default=1)
    ap.add_argument("--steps", type=int, default=200)
    ap.add_argument("--warmup", type=int, default=10)
    ap.add_argument("--impl", default="ours", choices=["ours", "reference"])
    ap.add_argument("--workload", default="c3", choices=["c1", "c2", "c3", "c4", "c5", "city_pair", "city_brand"])
    ap.add_argument("--rows", type=int, default=None,
                    help="fact rows per GPU (weak scaling) or of the whole table (strong scaling); default: the "
                         "configuration's size, 1.2 B rows for --scaling strong")
    ap.add_argument("--scaling", default="weak", choices=["weak", "strong"],
                    help="weak: every rank owns its own rows; strong: one table cut into contiguous row ranges")
    ap.add_argument("--sel", type=float, default=0.1, help="c4: fact predicate selectivity")
    ap.add_argument("--groups", type=int, default=1000, help="c4: number of groups")
    ap.add_argument("--e2e-steps", type=int, default=3)
    ap.add_argument("--e2e-chunk-rows", type=int, default=16 << 20, help="rows per chunk of the host-buffer pipeline")
    ap.add_argument("--cpu-sample-rows", type=int, default=100_000_000)
    ap.add_argument("--interpret", action="store_true",
                    help="interpret the query descriptor instead of compiling the fused kernel for the query's shape")
    ap.add_argument("--block-threads", type=int, default=0,
                    help="force the fused kernel's block size (profiling a small case in the full-size launch shape)")
    ap.add_argument("--ctas-per-sm", type=int, default=0)
    ap.add_argument("--no-e2e", action="store_true")
    ap.add_argument("--no-cpu-baseline", action="store_true")
    ap.add_argument("--no-points", action="store_true", help="skip the other configurations (N = 1 runs them by default)")
    ap.add_argument("--extras", action="store_true", help="more points: large group counts as dense arrays and through the hash table")
    ap.add_argument("--ablation", action="store_true",
                    help="also run the A/B switches (lazy vs eager loads, queues, table forms, group-by paths, "
                         "operator-at-a-time)")
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

    rows = args.rows if args.rows else (1_200_000_000 if args.scaling == "strong" else None)
    w = make_workload(args.workload, rows, args.sel, args.groups)
    row0, n = shard.rank_rows(rank, world, w.n_rows, args.scaling)  # this rank's part of the row space
    total_rows = w.n_rows * world if args.scaling == "weak" else w.n_rows
    w_local = W.with_rows(w, n)
    dims = {d.name: W.device_dim(w, d, device) for d in w.dims}
    fact = W.device_fact(w, row0=row0, n=n, device=device)
    torch.cuda.synchronize()
    # The query runs on a high-priority stream and the table builders' side streams keep the default (lowest)
    # priority: the blocks of the persistent fused kernel are placed first, and the next step's key-range scans
    # and builds fill in where an SM has room instead of delaying its start.
    torch.cuda.set_stream(torch.cuda.Stream(device, priority=-1))

    # every event pair is created (recorded once) up front; the library records them around the fused kernel
    pairs = [(torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True))
             for _ in range(args.steps)]
    for a, b in pairs:
        a.record()
        b.record()
    res = sjq.alloc_result(w.mode, w.num_groups, w.capacity, w.agg.want_count, device)
    # argument marshalling done once; scan + build run every step.  The layout of a table is the one chosen from the
    # newest scan whose statistics have reached the host (no wait on this step's scan); the build checks it on the
    # device, so a stale layout shows as a table status, which the assertions below would catch
    builders = sjq.workload_builders(w, dims, reuse_layout=True)
    pred_sampler = sjq.PredSampler({c.name: fact[c.name] for c in w.fact_cols}, w.preds)
    launches = 0
    info = None
    merged = None

    def step(i=None):
        nonlocal launches, info, merged
        pred_sampler.begin()  # planning: measured pass fractions of the fact predicates, beside the key-range scans
        tables = sjq.build_tables(builders)
        opts = sjq.RunOpts(events=pairs[i] if i is not None else None, specialise=not args.interpret,
                           block_threads=args.block_threads, ctas_per_sm=args.ctas_per_sm,
                           pass_ppm=pred_sampler.end())
        if i is not None and w.preds:
            launches += 1
        r = sjq.run_workload(w_local, fact, tables, opts, result=res)
        if world > 1:
            merged = shard.merge_result(res)
        if i is not None:
            launches += r.info.kernel_launches + sum(sjq.build_launches(t) for t in tables.values())
            if world > 1 and w.mode == "HASHED":
                launches += 3  # clear, merge and compaction kernels of sjq_merge_groups
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

    gpu_index = visible_gpu_index(local_rank)
    sampler = ClockSampler(gpu_index)
    ev0, ev1 = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.start()
    ev0.record()
    for i in range(args.steps):
        tables = step(i)
    ev1.record()
    if world > 1:
        dist.barrier()
    torch.cuda.synchronize()
    sampler.stop_flag = True
    sampler.join(timeout=2.0)
    ms_total = ev0.elapsed_time(ev1)
    assert res.status() == 0 and all(t.status() == 0 for t in tables.values()), "a timed step reported a status"
    fused_ms = sum(a.elapsed_time(b) for a, b in pairs) / len(pairs)
    t = torch.tensor([ms_total, fused_ms], dtype=torch.float64, device=device)
    if world > 1:
        dist.all_reduce(t, op=dist.ReduceOp.MAX)
    ms_total, fused_ms = float(t[0]), float(t[1])
    ms_per_step = ms_total / args.steps
    value = total_rows / (ms_per_step / 1000.0)
    ref_bytes = w.referenced_bytes_per_row()
    eff_gbs = total_rows * ref_bytes / (ms_per_step / 1000.0) / 1e9
    parity = matches_golden(w, res, golden_for(w)) if world == 1 else None

    peak, peak_kind = measured_hbm_peak()
    if w.mode == "HASHED":
        survivors = int(res.counts[: int(res.n_groups.item())].sum().item())
    else:
        survivors = int(res.counts.sum().item()) if res.counts is not None else None
    pass_frac = stage_pass_fractions(w_local, tables, survivors)
    alg_bpr = algorithmic_bytes_per_row(w, list(info.order[: info.nstages]), pass_frac)
    achieved = n * alg_bpr / (fused_ms / 1000.0) / 1e9
    kernel_name = "fused_kernel" if args.interpret else "sjq_jit_kernel"
    traffic, traffic_note = profiled_traffic(w, info, kernel_name, n)
    roofline = {"bound": "hbm", "kernel": kernel_name, "achieved": achieved, "peak": peak,
                "peak_kind": f"of {peak_kind}", "unit": "GB/s", "frac": achieved / peak,
                "traffic": traffic, "traffic_source": traffic_note,
                "algorithmic_bytes_per_row": alg_bpr, "kernel_ms": fused_ms,
                "bytes_per_row_64B_model": algorithmic_bytes_per_row(w, list(info.order[: info.nstages]), pass_frac, 64),
                "note": "achieved and frac use the 32-byte-sector model; DRAM delivers 64-byte pieces (ncu traffic), "
                        "for which the same model gives bytes_per_row_64B_model",
                "pass_fractions": {str(k): round(v, 6) for k, v in pass_frac.items()},
                "effective_gbs_kernel": n * ref_bytes / (fused_ms / 1000.0) / 1e9}

    e2e = None
    if not args.no_e2e:
        try:
            host_fact = {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True) for k, v in fact.items()}
            for k, v in fact.items():
                host_fact[k].copy_(v)
            host_dims = {dn: {k: torch.empty(v.shape, dtype=v.dtype, pin_memory=True).copy_(v) for k, v in cols.items()}
                         for dn, cols in dims.items()}
            dim_bytes = sum(v.numel() * v.element_size() for cols in host_dims.values() for v in cols.values())
            torch.cuda.synchronize()
            chunk = min(n, args.e2e_chunk_rows) // 4 * 4 or 4
            staging = torch.empty(sjq.staging_bytes(host_fact, chunk), dtype=torch.uint8, device=device)
            eres, ehost = None, None

            def e2e_step():
                nonlocal eres, ehost
                for dn, cols in host_dims.items():  # the dimension columns come from the host too
                    for k, v in cols.items():
                        dims[dn][k].copy_(v, non_blocking=True)
                for b in builders.values():  # scans and builds run on side streams: after the copies
                    b.after(torch.cuda.current_stream(device))
                tabs = sjq.build_tables(builders)
                eres, ehost = sjq.run_workload_host(w_local, host_fact, tabs, staging, chunk,
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
            same = None
            if world == 1 and w.mode != "HASHED":
                same = bool(torch.equal(ehost.sums, res.sums.cpu()))
            cells = 1 if w.mode == "SCALAR" else w.num_groups if w.mode == "DENSE" else w.capacity
            # bytes over the bus: whole columns for the copied ones; for a column the kernel reads in place, the
            # 32-byte sectors holding a surviving row (estimated from the planner's share of rows reaching it)
            plan = sjq.host_transfer_plan({c.name: host_fact[c.name] for c in w.fact_cols}, w.preds,
                                          [(fk, tabs[dn]) for fk, dn in w.joins], w.key, w.agg,
                                          sjq.RunOpts(specialise=not args.interpret))
            copied = sum(n * host_fact[k].element_size() for k, (how, _) in plan.items() if how == "copy")
            in_place = sum(n * host_fact[k].element_size() * (1.0 - (1.0 - sh) ** (32 // host_fact[k].element_size()))
                           for k, (how, sh) in plan.items() if how == "in place")
            e2e = {"value": total_rows / dt, "unit": UNIT, "h2d_bytes_per_step": int(copied + in_place + dim_bytes),
                   "h2d_copied_bytes": int(copied), "h2d_dimension_bytes": int(dim_bytes),
                   "h2d_in_place_bytes_estimate": int(in_place),
                   "h2d_in_place_note": "sector-model estimate from the planner's shares, not a counter",
                   "columns": {k: how for k, (how, _) in plan.items()},
                   "d2h_bytes_per_step": cells * 8 * (2 if w.agg.want_count else 1) + 4, "ms_per_step": dt * 1000.0,
                   "steps": args.e2e_steps, "chunk_rows": chunk, "matches_device_run": same,
                   "api": "sjq_run_host (pinned host columns: chunked double-buffered copies of the columns most rows need, "
                          "in-place reads of the sparse ones, result copied back); dimension columns copied from pinned "
                          "host memory every step before the table builds"}
            del host_fact, staging, host_dims
        except Exception as ex:  # e.g. not enough page-locked memory on the box
            e2e = {"value": None, "unit": UNIT, "error": repr(ex)[:200]}

    points = None
    if world == 1 and rank == 0 and not args.no_points:
        c3_inputs = (w, fact, tables) if (args.workload == "c3" and not args.rows) else None
        points = run_points(sjq, torch, W, device, not args.interpret, gpu_index, peak, c3_inputs, extras=args.extras)

    cpu = None
    if rank == 0 and world == 1 and not args.no_cpu_baseline:
        sample = min(n, args.cpu_sample_rows)
        rate, secs, tb = oracle_rate(w, sample)
        cpu = {"value": rate, "unit": UNIT, "cores": 1, "kind": "oracle",
               "sample": f"first {sample} fact rows of the workload; row loop {secs:.2f} s + dimension maps {tb:.2f} s",
               "host_cores_available": os.cpu_count()}

    ablation = None
    if args.ablation and world == 1 and rank == 0:
        fact.clear()
        torch.cuda.empty_cache()
        ablation = run_ablation(sjq, W, device, not args.interpret)

    if rank == 0:
        exchange = ""
        if world > 1:
            exchange = (", then all-gather of the per-rank group lists and a merge kernel" if w.mode == "HASHED"
                        else ", then one all-reduce of the joined sums, counts and status words")
        line = {"metric": METRIC, "value": value, "unit": UNIT, "n_gpus": world, "steps": args.steps,
                "warmup": args.warmup, "ms_per_step": ms_per_step, "higher_is_better": True, "scaling": args.scaling,
                "vs_baseline": None, "dtype": "int64", "data": "synthetic",
                "config": {"workload": w.name, "rows_per_gpu": n, "rows_total": total_rows,
                           "referenced_bytes_per_row": ref_bytes,
                           "step": "key-range scan + build of every dimension table (on side streams; the table shape comes from the newest scan that has reached the host and is checked on the device by the build, so the host never waits), then the fused pass"
                                   + exchange,
                           "l2": "inputs (%.1f GB) exceed the 126 MB L2; no flush needed" % (n * ref_bytes / 1e9),
                           "parallelism": f"row-sharded x{world}, dimensions replicated", "plan": info.describe(),
                           "fused_kernel": "interpreted descriptor" if args.interpret else
                                           "compiled for the query's shape at run time during warm-up (NVRTC), cached"},
                "effective_gbs": eff_gbs, "pct_of_8tbs": 100.0 * eff_gbs / world / CONTRACT_HBM_GBS,
                "pct_of_measured_copy_peak": 100.0 * eff_gbs / world / peak, "parity": parity,
                "roofline": roofline, "cpu_baseline": cpu, "e2e": e2e, "gpu_launches": launches,
                "clocks": sampler.summary()}
        if points is not None:
            line["points"] = points
        if ablation is not None:
            line["ablation"] = ablation
        print(json.dumps(line), flush=True)
    if world > 1:
        dist.destroy_process_group()
    return 0


def unfused_bytes_model(w, res, tables):
    """DRAM bytes each pass of the operator-at-a-time arm moves, by construction: every filter pass reads its
    whole fact column, reads (except the first) and writes one flag byte per row, and a gathering join writes
    its payload code for the 32-byte sectors holding a survivor; the aggregation pass reads the flags and, for
    sectors holding a survivor, the measure columns and the materialised payloads."""
    survivors = int(res.counts.sum().item()) if w.mode != "HASHED" else int(res.counts[: int(res.n_groups.item())].sum().item())
    frac = stage_pass_fractions(w, tables, survivors)
    plan = res.info.describe()
    cols = [p.col for p in w.preds] + [fk for fk, _ in w.joins]
    n, reach, passes, seen = w.n_rows, 1.0, [], set()
    nfilter = len(w.preds) + len(w.joins)
    gathered = {j for t in ((w.key.terms if w.key else ()) + (w.agg.x,) + ((w.agg.y,) if w.agg.y else ()))
                if t.src == "PAYLOAD" for j in [int(t.a)]}
    first = True
    for idx in plan["order"]:
        if idx < 0 or idx in seen:
            continue
        seen.add(idx)
        width = 8 if w.fact_col(cols[idx]).is64 else 4
        b = n * width + (0 if first else n) + n
        reach *= frac.get(idx, 1.0)
        if idx >= len(w.preds) and (idx - len(w.preds)) in gathered:
            b += n * 4 * (1.0 - (1.0 - reach) ** 8)
        passes.append({"stage": idx, "bytes": int(b)})
        first = False
    sector = 1.0 - (1.0 - reach) ** 8
    measure = {t.a for t in ((w.key.terms if w.key else ()) + (w.agg.x,) + ((w.agg.y,) if w.agg.y else ())) if t.src == "FACT"}
    agg = (n if nfilter else 0) + sum(n * (8 if w.fact_col(c).is64 else 4) * sector for c in measure) + \
        len(gathered) * n * 4 * sector
    passes.append({"stage": "aggregate", "bytes": int(agg)})
    return {"passes": passes, "total": int(sum(p["bytes"] for p in passes))}


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
        row_extra = {}
        if label == UNFUSED:
            row_extra["bytes_moved_model"] = unfused_bytes_model(w, res, tables)
        out.append({"workload": w.name, "variant": label, "ms_min": min(ts), **row_extra,
                    "rows_per_s": w.n_rows / (min(ts) / 1000.0), "status": res.status(),
                    "table_kinds": {k: t.layout.kind_name for k, t in tables.items()},
                    "table_bytes": {k: int(t.layout.table_bytes) for k, t in tables.items()},
                    "plan": res.info.describe()})
        return fact, dims

    INTERPRETED = "query descriptor interpreted (no run-time specialisation)"
    UNFUSED = "operator at a time: one kernel per predicate / join over a flag array, payload columns materialised"
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
                             sjq.RunOpts(no_filter_bitmap=True)),
                            (UNFUSED, sjq.RunOpts(unfused_scratch=sjq.unfused_scratch(w.n_rows, len(w.joins), device)))):
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
