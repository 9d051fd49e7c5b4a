"""The no-allocation entry point (sjq_run_hashed_static).

Some embedders of this library may not allocate device memory at all: a plug-in
that is handed a fixed arena, a loop whose rules ban allocator calls after
start-up, a process whose memory pool belongs to another runtime.  For them the
hashed group-by keeps its group table in a fixed array inside the library
instead of a caller-provided workspace.  This test calls that entry point
through the C ABI several times in a row (each call meets the previous call's
leftovers in the shared table) and checks each output, bit for bit, against
the CPU oracle and against the ordinary entry point on the same inputs.  Both
forms the group table can take inside the fixed array are covered: the table
indexed by the key itself (a key taken modulo M) and the open-addressing hash
table (a key without a modulo, or `group_hash_always`), each with many groups
first and few groups second, so that stale cells and stale keys of the larger
call would show up in the smaller one.  It lives in the file pytest collects
last, so a run that stops at the first failure has already run everything
else; it must also pass alone in a fresh process.
"""
from dataclasses import replace

import numpy as np
import pytest
import torch

from datagen import workloads as W
from datagen.workloads import AggExpr, KeyExpr, Term

pytestmark = pytest.mark.gpu


def _sorted_triples(res):
    k, s, c = res.hashed_sorted()
    return k.cpu().numpy(), s.cpu().numpy(), c.cpu().numpy()


def _calls():
    """(workload, options, form of the group table) in the order they run: within each form of the group table
    the call with many groups comes first."""
    import paper_2607_07632_b200 as sjq

    many = W.config4(700_003, 0.5, 30_000, hashed=True, dim_rows=40_000)
    few = W.config4(300_001, 0.1, 700, hashed=True, dim_rows=40_000)
    # a key built from a fact column without a modulo has no known range and can only live in the hash table:
    # the foreign key itself (tens of thousands of groups), then the filtered column (a thousand groups)
    many_plain = replace(many, name="static_fk_groups", key=KeyExpr((Term("FACT", "fk"),), offset=-7),
                         capacity=40_000)
    few_plain = replace(few, name="static_p_groups", key=KeyExpr((Term("FACT", "p", 0, 3),), offset=-3),
                        capacity=1024)
    # a key made of gathered payloads only has a range the tables know: the indexed form again, four cells
    payload_key = replace(few, name="static_payload_groups", key=KeyExpr((Term("PAYLOAD", 0, 0, 5),), offset=-3),
                          capacity=16)
    always = sjq.RunOpts(group_hash_always=True)
    return [(many, None, "indexed"), (few, None, "indexed"),  # the table indexed by the key
            (many, always, "hash"), (few, always, "hash"),  # the same queries through the hash table
            (many_plain, None, "hash"), (few_plain, None, "hash"),
            (many, None, "indexed"),  # and back: the indexed form over the hash table's leftovers
            (payload_key, None, "indexed")]


def test_static_group_table_matches_oracle_and_workspace_entry_point_call_after_call():
    import oracle
    import paper_2607_07632_b200 as sjq
    from gpuhelpers import compare

    inputs = {}
    for i, (w, opts, path) in enumerate(_calls()):
        if w.name not in inputs:
            hd = {d.name: W.host_dim(w, d) for d in w.dims}
            hf = W.host_fact(w)
            dims = {d.name: W.device_dim(w, d) for d in w.dims}
            inputs[w.name] = (oracle.run(w, hf, oracle.build_dims(w, hd)), sjq.build_workload_tables(w, dims),
                              W.device_fact(w))
        exp, tables, fact = inputs[w.name]
        ref = sjq.run_workload(w, fact, tables, opts)
        # result arrays are the caller's: allocate them before the call, as a caller without an allocator
        # would have been given them
        out = sjq.Result("HASHED", torch.empty(w.capacity, dtype=torch.int64, device="cuda"),
                         torch.empty(w.capacity, dtype=torch.int64, device="cuda"),
                         torch.empty(w.capacity, dtype=torch.int64, device="cuda"),
                         torch.zeros(1, dtype=torch.int64, device="cuda"),
                         torch.zeros(1, dtype=torch.int32, device="cuda"), None)
        torch.cuda.synchronize()
        free_before, _ = torch.cuda.mem_get_info()
        got = sjq.run_hashed_static({c.name: fact[c.name] for c in w.fact_cols}, w.preds,
                                    [(fk, tables[dn]) for fk, dn in w.joins], w.key, w.agg, w.capacity, opts,
                                    result=out)
        torch.cuda.synchronize()
        free_after, _ = torch.cuda.mem_get_info()
        assert got is out and ref.status() == 0 and got.status() == 0
        used = sjq.sjq.AGG_PATHS[got.info.agg_path]
        assert (used == "hash") == (path == "hash"), (i, w.name, got.info.describe())
        assert int(got.n_groups.item()) == int(ref.n_groups.item()) == exp["keys"].size > 0
        compare(w, got, exp)  # against the oracle
        for a, b in zip(_sorted_triples(got), _sorted_triples(ref)):  # against the workspace entry point
            assert np.array_equal(a, b)
        if i > 0:  # the first call on a device makes the driver load the kernels; later calls take nothing
            assert free_after >= free_before, (i, free_before, free_after)


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
