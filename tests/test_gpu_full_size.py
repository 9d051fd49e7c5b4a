"""Parity at the benchmark's full sizes, in the launch configurations bench.py
times (the fused kernel compiled for the query's shape, which is its default,
and the interpreted descriptor; inputs generated on the device): each result must equal,
bit for bit, the expected values the CPU oracle wrote to tests/golden/full_*.json
(tests/golden/make_full_size.py).  Hashed results are compared through the
SHA-256 of their (key, sum, count) triples in ascending key order."""
import hashlib
import json
import os

import numpy as np
import pytest
import torch

from datagen import workloads as W

pytestmark = pytest.mark.gpu
GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def _golden(tag):
    path = os.path.join(GOLDEN, f"full_{tag}.json")
    if not os.path.exists(path):
        pytest.skip(f"{path} not generated")
    with open(path) as f:
        return json.load(f)


def _run(w):
    import paper_2607_07632_b200 as sjq

    dims = {d.name: W.device_dim(w, d) for d in w.dims}
    tables = sjq.build_workload_tables(w, dims)
    fact = W.device_fact(w)
    results = []
    variants = [sjq.RunOpts(specialise=True), sjq.RunOpts(specialise=False)]
    if w.mode == "HASHED":  # the group hash table as well as the direct-indexed table a modulo key allows
        variants.append(sjq.RunOpts(specialise=True, group_hash_always=True))
    for opts in variants:
        res = sjq.run_workload(w, fact, tables, opts)
        torch.cuda.synchronize()
        assert res.status() == 0 and all(t.status() == 0 for t in tables.values())
        results.append(res)
    entries = {k: t.layout.entries for k, t in tables.items()}
    del fact
    torch.cuda.empty_cache()
    return results, entries


def _check(w, tag):
    g = _golden(tag)
    assert g["rows"] == w.n_rows and g["workload"] == w.name
    results, entries = _run(w)
    assert entries == g["dim_entries"]
    for res in results:
        _compare(w, g, res)


def _compare(w, g, res):
    if w.mode == "SCALAR":
        assert int(res.sums[0].item()) == g["sum"] and int(res.counts[0].item()) == g["count"]
    elif w.mode == "DENSE":
        assert res.sums.cpu().tolist() == g["sums"]
        assert res.counts.cpu().tolist() == g["counts"]
    else:
        k, s, c = res.hashed_sorted()
        k, s, c = k.cpu().numpy(), s.cpu().numpy(), c.cpu().numpy()
        assert k.size == g["groups"] and int(s.sum()) == g["total_sum"] and int(c.sum()) == g["total_count"]
        h = hashlib.sha256()
        for a in (k, s, c):
            h.update(np.ascontiguousarray(a, dtype="<i8").tobytes())
        assert h.hexdigest() == g["sha256"]


@pytest.mark.parametrize("name", ["c1", "c2", "c3", "c5"])
def test_full_size_config(name):
    _check(W.CONFIGS[name](), name)


@pytest.mark.parametrize("sel", list(W.C4_THRESHOLDS))
@pytest.mark.parametrize("groups", W.C4_GROUPS)
def test_full_size_sweep_point(sel, groups):
    _check(W.config4(600_000_000, sel, groups), f"c4_s{sel:g}_g{groups}")


def test_more_than_2_pow_32_rows_equals_split_runs():
    """Maximum-size edge: beyond 2^32 rows the survivor queues switch to tile-relative offsets and are
    drained per tile.  The oracle cannot hold such a table, so the check is the split-and-add property
    (pinned for the oracle on the CPU): one run over all rows must equal two accumulated runs over
    halves that each stay below 2^32 rows, and the count must equal the closed form of the generator."""
    import paper_2607_07632_b200 as sjq
    from datagen import UNIFORM_I32, fill_device
    from datagen.workloads import AggExpr, KeyExpr, Pred, Term

    n = (1 << 32) + 4099
    free, _ = torch.cuda.mem_get_info()
    if free < n * 4 + (2 << 30):
        pytest.skip("not enough device memory for a 17 GB column")
    p = fill_device(UNIFORM_I32, 20260707, 901, 0, n, 0, 9999)
    fact = {"p": p}
    half = 1 << 31
    parts = ({"p": p[:half]}, {"p": p[half:]})
    for kw in (dict(mode="SCALAR", key=None),
               dict(mode="DENSE", key=KeyExpr((Term("FACT", "p"),), modulo=7), num_groups=7)):
        agg = AggExpr("COL", Term("FACT", "p"))
        preds = (Pred("p", "LT", 2500),)
        acc = sjq.run(parts[0], preds, (), agg=agg, **kw)
        acc = sjq.run(parts[1], preds, (), agg=agg, opts=sjq.RunOpts(accumulate=True), result=acc, **kw)
        for specialise in (False, True):
            whole = sjq.run(fact, preds, (), agg=agg, opts=sjq.RunOpts(specialise=specialise), **kw)
            torch.cuda.synchronize()
            assert whole.status() == 0 and acc.status() == 0
            assert torch.equal(whole.sums, acc.sums) and torch.equal(whole.counts, acc.counts)
            assert int(whole.counts.sum().item()) == int((p < 2500).sum().item())
    del p, fact, parts
    torch.cuda.empty_cache()
