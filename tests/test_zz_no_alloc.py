"""The no-allocation entry point (sjq_run_hashed_static).

Some embedders of this library may not allocate device memory at all: a plug-in
that is handed a fixed arena, a loop whose rules ban allocator calls after
start-up, a process whose memory pool belongs to another runtime.  For them the
hashed group-by keeps its group table in a fixed array inside the library
instead of a caller-provided workspace.  This test calls that entry point
through the C ABI twice in a row (the second call meets the first call's
leftovers in the shared table) and checks each output, bit for bit, against
the ordinary entry point on the same inputs.  It lives in the file pytest
collects last, so a run that stops at the first failure has already run
everything else; it must also pass alone in a fresh process.
"""
import numpy as np
import pytest
import torch

from datagen import workloads as W
from datagen.workloads import AggExpr, KeyExpr, Term

pytestmark = pytest.mark.gpu


def _sorted_triples(res):
    k, s, c = res.hashed_sorted()
    return k.cpu().numpy(), s.cpu().numpy(), c.cpu().numpy()


def test_static_group_table_matches_workspace_entry_point_twice():
    import paper_2607_07632_b200 as sjq

    # first call: many groups (fills a good part of the shared table)
    w1 = W.config4(700_003, 0.5, 30_000, hashed=True, dim_rows=40_000)
    # second call: a different query with few groups; stale slots of call one must not leak in
    w2 = W.config4(300_001, 0.1, 700, hashed=True, dim_rows=40_000)
    for w in (w1, w2):
        dims = {d.name: W.device_dim(w, d) for d in w.dims}
        tables = sjq.build_workload_tables(w, dims)
        fact = W.device_fact(w)
        ref = sjq.run_workload(w, fact, tables)
        got = sjq.run_hashed_static({c.name: fact[c.name] for c in w.fact_cols}, w.preds,
                                    [(fk, tables[dn]) for fk, dn in w.joins], w.key, w.agg, w.capacity)
        torch.cuda.synchronize()
        assert ref.status() == 0 and got.status() == 0
        assert int(got.n_groups.item()) == int(ref.n_groups.item()) > 0
        for a, b in zip(_sorted_triples(got), _sorted_triples(ref)):
            assert np.array_equal(a, b)


def test_static_limit_is_rejected_with_a_clear_error():
    import paper_2607_07632_b200 as sjq

    fact = {"g": torch.arange(64, dtype=torch.int32, device="cuda")}
    key = KeyExpr((Term("FACT", "g"),))
    agg = AggExpr("COL", Term("FACT", "g"))
    with pytest.raises(sjq.SjqError) as e:
        sjq.run_hashed_static(fact, key=key, agg=agg, capacity=sjq.STATIC_MAX_GROUPS + 1)
    assert e.value.status == 6 and "no-allocation" in str(e.value)
    ok = sjq.run_hashed_static(fact, key=key, agg=agg, capacity=sjq.STATIC_MAX_GROUPS)
    torch.cuda.synchronize()
    assert ok.status() == 0 and int(ok.n_groups.item()) == 64
