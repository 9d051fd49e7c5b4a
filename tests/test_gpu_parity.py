"""Parity of the CUDA path (through the C ABI) with the CPU oracle: bit-exact
on every output element, on the same seeded inputs."""
from dataclasses import replace

import numpy as np
import pytest
import torch

import oracle
from datagen import workloads as W
from datagen.workloads import AggExpr, KeyExpr, Pred, Term

pytestmark = pytest.mark.gpu

sjq = pytest.importorskip("paper_2607_07632_b200") if torch.cuda.is_available() else None

from gpuhelpers import compare, oracle_result, run_both, to_dev  # noqa: E402
from qhelpers import adhoc, ex1, ex2, ex3, random_query  # noqa: E402
from bruteforce import dup_keys_among_passing  # noqa: E402

RAGGED = [0, 1, 3, 4, 5, 255, 256, 257, 2047, 2048, 2049, 4097, 100003]


def test_hand_examples():
    for mk in (ex1, ex2, ex3):
        w, fact, hd, _ = mk()
        res, exp, _ = run_both(w, fact, hd)
        assert res.status() == 0
        compare(w, res, exp)


@pytest.mark.parametrize("seed", range(200))
def test_random_small_queries(seed):
    w, fact, hd = random_query(seed, allow_dup=False, wide_keys=True)
    res, exp, _ = run_both(w, fact, hd, check=False)
    if exp["status"] == oracle.GROUP_RANGE:
        assert res.status() == 18
        # rows with an in-range key still land where the oracle puts them
        compare(w, res, exp)
    else:
        assert res.status() == 0
        compare(w, res, exp)


@pytest.mark.parametrize("seed", range(200, 240))
def test_random_queries_option_matrix(seed):
    w, fact, hd = random_query(seed, n_fact=700, allow_dup=False, wide_keys=True)
    dev_fact = to_dev(fact)
    tables = None
    for opts in (sjq.RunOpts(), sjq.RunOpts(eager_loads=True), sjq.RunOpts(smem_tables=1),
                 sjq.RunOpts(block_threads=128, ctas_per_sm=1), sjq.RunOpts(block_threads=256, compaction=2, smem_tables=1), sjq.RunOpts(agg_path=2),
                 sjq.RunOpts(compaction=2), sjq.RunOpts(compaction=1), sjq.RunOpts(no_filter_bitmap=True),
                 sjq.RunOpts(group_hash_always=True), sjq.RunOpts(warp_agg=1), sjq.RunOpts(warp_agg=1, agg_path=2),
                 sjq.RunOpts(hot_keys=1), sjq.RunOpts(hot_keys=1, compaction=1),
                 sjq.RunOpts(unfused_scratch=sjq.unfused_scratch(w.n_rows, len(w.joins))),
                 sjq.RunOpts(order=tuple(reversed(range(len(w.preds) + len(w.joins)))))):
        res, exp, tables = run_both(w, fact, hd, opts=opts, check=False, dev_fact=dev_fact, tables=tables)
        assert (res.status() == 18) == (exp["status"] == oracle.GROUP_RANGE)
        compare(w, res, exp)


@pytest.mark.parametrize("n", RAGGED)
@pytest.mark.parametrize("cfg", ["c1", "c2", "c3", "c4d", "c4h", "c5"])
def test_configs_ragged_sizes(cfg, n):
    w = {"c1": lambda: W.config1(n), "c2": lambda: W.config2(n), "c3": lambda: W.config3(n),
         "c4d": lambda: W.config4(n, 0.5, 1000, dim_rows=50000),
         "c4h": lambda: W.config4(n, 0.5, 100000, dim_rows=50000),
         "c5": lambda: W.config5(n, 20000)}[cfg]()
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, _ = run_both(w, fact, hd)
    assert res.status() == 0
    compare(w, res, exp)


@pytest.mark.parametrize("mk", [lambda: W.config1(1_500_007), lambda: W.config2(2_000_003),
                                lambda: W.config3(2_500_001), lambda: W.config5(1_200_005, 300000)] +
                         [lambda s=s, g=g: W.config4(1_000_003, s, g) for s in (0.0001, 0.1, 1.0)
                          for g in (1, 1000, 100000, 1000000)])
def test_configs_multi_tile(mk):
    w = mk()
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, tables = run_both(w, fact, hd)
    assert res.status() == 0
    compare(w, res, exp)
    # the same query with every switch flipped gives the same bits
    dev_fact = to_dev(fact)
    for opts in (sjq.RunOpts(eager_loads=True, smem_tables=1, compaction=1),
                 sjq.RunOpts(agg_path=2 if w.mode == "DENSE" else 0, block_threads=256, compaction=2)):
        res2, _, _ = run_both(w, fact, hd, opts=opts, dev_fact=dev_fact, tables=tables)
        compare(w, res2, exp)


def test_device_generator_matches_host():
    for w in (W.config1(100_003), W.config3(100_003), W.config5(100_003, 50000)):
        host = W.host_fact(w)
        dev = W.device_fact(w)
        for k in host:
            assert np.array_equal(dev[k].cpu().numpy(), host[k]), (w.name, k)
        # a window in the middle of a large table is the same function of the row
        dev2 = W.device_fact(w, 50_000, 1000)
        for k in host:
            assert np.array_equal(dev2[k].cpu().numpy(), host[k][50_000:51_000])
        for d in w.dims:
            hd, dd = W.host_dim(w, d), W.device_dim(w, d)
            for k in hd:
                assert np.array_equal(dd[k].cpu().numpy(), hd[k])


def test_table_kinds_and_sizes():
    # Section 3.3 sizes: 3M keys -> 3 MB byte-packed map (12 MB as int32)
    w = W.config3(10)
    dims = {d.name: W.device_dim(w, d) for d in w.dims}
    tabs = sjq.build_workload_tables(w, dims)
    # with byte-or-wider codes, as in the paper: the 3 MB customer map
    L = sjq.build_dim(dims["customer"], "custkey", w.dim("customer").preds, ("nation",), min_code_bits=8).layout
    # the key range is taken among the rows passing the filter
    assert L.kind_name == "DIRECT_U8" and 2_999_000 <= L.slots <= 3_000_000 and L.code_bits == 8
    # byte-packed codes plus the presence bitmap over the same slots (an eighth of a byte per slot)
    assert L.filter_bits >= L.slots and L.filter_bits % 128 == 0
    assert L.slots + L.slots // 8 <= L.table_bytes <= 3_000_000 + 375_000 + 1024
    # by default the five nations of the region (codes 0..4, 0xF = filtered out) take four bits: half of that
    L = tabs["customer"].layout
    assert L.kind_name == "DIRECT_U4" and L.code_bits == 4 and L.pay_bits[0] == 3
    assert L.slots // 2 + L.slots // 8 <= L.table_bytes <= 1_500_000 + 375_000 + 1024
    assert tabs["supplier"].layout.kind_name == "DIRECT_BITMAP" and 199_900 <= tabs["supplier"].layout.slots <= 200_000
    assert tabs["part"].layout.kind_name == "DIRECT_BITMAP"
    d = tabs["date"].layout  # two years: one payload bit, the marker needs a second
    assert d.kind_name == "DIRECT_U2" and d.entries == 729 and d.kmin == 19970101 and d.kmax == 19981230
    # an unfiltered dimension with contiguous keys holds every key of its range: no marker, the range test decides
    w4 = W.config4(10)
    t4 = sjq.build_workload_tables(w4, {x.name: W.device_dim(w4, x) for x in w4.dims})["dim"]
    assert t4.layout.kind_name == "DIRECT_U2" and t4.layout.entries == t4.layout.slots == 3_000_000
    assert t4.layout.pay_max[0] - t4.layout.pay_min[0] == 3 and t4.check().status() == 0
    # forcing the unpacked form: open addressing at load <= 0.5
    t = sjq.build_dim(dims["customer"], "custkey", w.dim("customer").preds, ("nation",), force_kind=sjq.sjq.FORCE_HASH)
    assert t.layout.kind_name == "HASH_I32" and t.layout.slots >= 2 * t.layout.entries
    assert t.check().status() == 0
    # wide payloads choose wider codes
    cols = {"k": torch.arange(1, 1001, dtype=torch.int32, device="cuda"),
            "a": torch.arange(0, 1000, dtype=torch.int32, device="cuda") * 70,
            "b": torch.arange(0, 1000, dtype=torch.int32, device="cuda") - 500}
    assert sjq.build_dim(cols, "k", (), ("a",)).layout.kind_name == "DIRECT_U32"
    assert sjq.build_dim(cols, "k", (), ("b",)).layout.kind_name == "DIRECT_U16"
    t2 = sjq.build_dim(cols, "k", (), ("a", "b"))
    assert t2.layout.kind_name == "DIRECT_U32" and t2.layout.pay_bits[0] == 17 and t2.layout.pay_bits[1] == 10


def test_duplicate_key_is_reported():
    for force in (0, sjq.sjq.FORCE_HASH):
        for npay in (0, 1):
            cols = {"k": torch.tensor([5, 9, 7, 9], dtype=torch.int32, device="cuda"),
                    "p": torch.tensor([1, 2, 3, 4], dtype=torch.int32, device="cuda")}
            t = sjq.build_dim(cols, "k", (), ("p",)[:npay], force_kind=force)
            assert t.status() == 16
            # the duplicate filtered away -> fine
            t = sjq.build_dim(cols, "k", (Pred("p", "NE", 4),), ("p",)[:npay], force_kind=force)
            assert t.status() == 0


@pytest.mark.parametrize("wide", [False, True])
def test_undersized_hash_table_reports_table_full(wide):
    """A consistent layout with too few slots for the rows that pass (a stale plan, a caller's own
    sizing): the bounded insert loop gives up and the status word says TABLE_FULL; nothing is written
    outside the (smaller) table and the context stays usable."""
    dt = torch.int64 if wide else torch.int32
    cols = {"k": torch.arange(1, 1001, dtype=dt, device="cuda") * 7919,
            "p": torch.arange(0, 1000, dtype=torch.int32, device="cuda")}

    def shrink(L):
        assert L.kind_name == ("HASH_I64" if wide else "HASH_I32")
        L.slots = 80  # whole buckets for every key and code width
        L.table_bytes = sjq.layout_bytes(L)

    for pay in ((), ("p",)):
        t = sjq.build_dim(cols, "k", (), pay, force_kind=sjq.sjq.FORCE_HASH, edit_layout=shrink)
        assert t.status() == 17 and "full" in sjq.strerror(17)
        # exactly as many rows as slots still fit
        t = sjq.build_dim(cols, "k", (Pred("p", "LT", 80),), pay, force_kind=sjq.sjq.FORCE_HASH, edit_layout=shrink)
        assert t.status() == 0
        t = sjq.build_dim(cols, "k", (Pred("p", "LT", 81),), pay, force_kind=sjq.sjq.FORCE_HASH, edit_layout=shrink)
        assert t.status() == 17
    assert sjq.build_dim(cols, "k", (), ("p",), force_kind=sjq.sjq.FORCE_HASH).status() == 0


def test_sub_byte_tables_with_and_without_the_miss_marker():
    """2- and 4-bit codes.  A dimension that holds every key of its range uses all code values and lets the
    range test decide a hit; any other keeps all-ones as the miss marker.  Keys outside the range, keys
    filtered out and duplicate keys behave as for the byte-wide maps, and a layout that promises "every key"
    for data that lacks one is reported, not followed."""
    import ctypes

    rng = np.random.default_rng(7)
    n = 4099
    for width, hi in ((2, 3), (4, 15)):
        keys = np.arange(100, 100 + 577, dtype=np.int32)
        dim = {"k": keys, "w": rng.integers(0, hi + 1, keys.size).astype(np.int32), "f": (keys % 3).astype(np.int32)}
        dim["w"][:hi + 1] = np.arange(hi + 1)  # every code value occurs, all-ones included
        fact = {"fk": rng.integers(60, 720, n).astype(np.int32), "m": rng.integers(0, 1000, n).astype(np.int32)}
        for preds, full in (([], True), ([Pred("f", "NE", 0)], False)):
            w = adhoc("sub", fact, [("d", dim, "k", preds, ["w"])], [("fk", "d")], [],
                      KeyExpr((Term("PAYLOAD", 0, 0),)), AggExpr("ADD", Term("FACT", "m"), Term("PAYLOAD", 0, 0, 7)),
                      "DENSE", num_groups=hi + 1)
            for opts in (None, sjq.RunOpts(specialise=True), sjq.RunOpts(compaction=1),
                         sjq.RunOpts(specialise=True, pass_ppm=(990_000,)), sjq.RunOpts(smem_tables=1),
                         sjq.RunOpts(no_filter_bitmap=True)):
                res, exp, tabs = run_both(w, fact, {"d": dim}, opts=opts)
                L = tabs["d"].layout
                # without the marker the narrow width holds all values; with it the next width is needed
                assert L.kind_name == (f"DIRECT_U{width}" if full else {2: "DIRECT_U4", 4: "DIRECT_U8"}[width])
                assert (L.entries == L.slots) == full and res.status() == 0
                compare(w, res, exp)
    # duplicate key in a sub-byte table
    cols = {"k": torch.tensor([5, 6, 7, 6], dtype=torch.int32, device="cuda"),
            "p": torch.tensor([1, 2, 0, 1], dtype=torch.int32, device="cuda")}
    assert sjq.build_dim(cols, "k", (), ("p",)).status() == 16
    # a layout planned for the full dimension, used to build from data that lacks a key
    full_cols = {"k": torch.arange(1, 101, dtype=torch.int32, device="cuda"),
                 "p": torch.arange(0, 100, dtype=torch.int32, device="cuda") % 4}
    planned = sjq.build_dim(full_cols, "k", (), ("p",))
    assert planned.layout.kind_name == "DIRECT_U2" and planned.status() == 0

    def stale(L):
        ctypes.memmove(ctypes.byref(L), ctypes.byref(planned.layout), ctypes.sizeof(L))

    assert sjq.build_dim(full_cols, "k", (Pred("k", "NE", 50),), ("p",), edit_layout=stale).status() == 21


def test_reserved_key_and_empty_dimension():
    cols = {"k": torch.tensor([-(2 ** 63), 4], dtype=torch.int64, device="cuda")}
    assert sjq.build_dim(cols, "k", force_kind=sjq.sjq.FORCE_HASH).status() == 20
    fact = {"fk": np.array([4, 5, -(2 ** 63)], np.int64), "v": np.array([1, 2, 3], np.int32)}
    dim = {"k": np.array([4, 5], np.int64), "f": np.array([0, 0], np.int32)}
    w = adhoc("empty", fact, [("d", dim, "k", [Pred("f", "EQ", 1)], [], True)], [("fk", "d")], [], None,
              AggExpr("COL", Term("FACT", "v")), "SCALAR")
    res, exp, tabs = run_both(w, fact, {"d": dim})
    assert tabs["d"].layout.entries == 0
    compare(w, res, exp)
    assert int(res.counts[0].item()) == 0


def test_fk_outside_key_range_is_a_miss():
    fact = {"fk": np.array([-7, 0, 1, 5, 6, 2 ** 31 - 1, -2 ** 31], np.int32), "v": np.arange(7, dtype=np.int32) + 1}
    dim = {"k": np.array([1, 5], np.int32), "p": np.array([3, 4], np.int32)}
    for force in (False, True):
        w = adhoc("miss", fact, [("d", dim, "k", [], ["p"], force)], [("fk", "d")], [], None,
                  AggExpr("MUL", Term("FACT", "v"), Term("PAYLOAD", 0, 0)), "SCALAR")
        res, exp, _ = run_both(w, fact, {"d": dim})
        compare(w, res, exp)
        assert int(res.sums[0].item()) == 25


def test_hashed_overflow_and_group_range_status():
    n = 5000
    fact = {"g": np.arange(n, dtype=np.int32)}
    w = adhoc("ovf", fact, [], [], [], KeyExpr((Term("FACT", "g"),)), AggExpr("COL", Term("FACT", "g")), "HASHED",
              capacity=64)
    res = sjq.run_workload(w, to_dev(fact), {})
    assert res.status() == 19
    w = adhoc("rng", fact, [], [], [], KeyExpr((Term("FACT", "g"),)), AggExpr("COL", Term("FACT", "g")), "DENSE",
              num_groups=100)
    res = sjq.run_workload(w, to_dev(fact), {})
    assert res.status() == 18
    assert int(res.counts.sum().item()) == 100


def test_accumulate_equals_whole():
    w = W.config3(300_001)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, tables = run_both(w, fact, hd)
    k = 123_457
    a = to_dev({c: v[:k] for c, v in fact.items()})
    b = to_dev({c: v[k:].copy() for c, v in fact.items()})
    r = sjq.run_workload(replace(w, n_rows=k), a, tables)
    r = sjq.run_workload(replace(w, n_rows=w.n_rows - k), b, tables, sjq.RunOpts(accumulate=True), result=r)
    torch.cuda.synchronize()
    compare(w, r, exp)


def test_invalid_arguments_are_rejected():
    fact = {"a": torch.zeros(8, dtype=torch.int32, device="cuda"), "b": torch.zeros(9, dtype=torch.int32, device="cuda")}
    with pytest.raises(sjq.SjqError) as e:
        sjq.run(fact, agg=AggExpr("COL", Term("FACT", "a")))
    assert e.value.status == 1
    ok = {"a": torch.zeros(64, dtype=torch.int32, device="cuda")}
    with pytest.raises(sjq.SjqError) as e:  # misaligned column
        sjq.run({"a": ok["a"][1:9]}, agg=AggExpr("COL", Term("FACT", "a")))
    assert e.value.status == 3
    with pytest.raises(sjq.SjqError) as e:  # grouped mode without a key
        sjq.run(ok, agg=AggExpr("COL", Term("FACT", "a")), mode="DENSE", num_groups=4)
    assert e.value.status == 1
    dim = sjq.build_dim({"k": torch.arange(4, dtype=torch.int64, device="cuda")}, "k")
    with pytest.raises(sjq.SjqError) as e:  # int32 fk into an int64-keyed table
        sjq.run(ok, joins=[("a", dim)], agg=AggExpr("COL", Term("FACT", "a")))
    assert e.value.status == 2


def test_host_buffer_entry_point_matches_oracle():
    for w in (W.config3(1_000_003), W.config4(500_001, 0.5, 100000, dim_rows=50000), W.config1(300_001)):
        fact = W.host_fact(w)
        hd = {d.name: W.host_dim(w, d) for d in w.dims}
        res, exp, tables = run_both(w, fact, hd)
        host_fact = {k: torch.from_numpy(v).pin_memory() for k, v in fact.items()}
        chunk = 65536 * 3  # several chunks and a ragged last one
        staging = torch.empty(sjq.staging_bytes(host_fact, chunk), dtype=torch.uint8, device="cuda")
        r, h = sjq.run_workload_host(w, host_fact, tables, staging, chunk)
        torch.cuda.synchronize()
        assert int(h.status[0]) == 0
        compare(w, r, exp)
        if w.mode == "SCALAR":
            assert int(h.sums[0]) == exp["sum"] and int(h.counts[0]) == exp["count"]
        elif w.mode == "DENSE":
            assert np.array_equal(h.sums.numpy(), exp["sums"]) and np.array_equal(h.counts.numpy(), exp["counts"])
        else:
            n = int(h.n_groups[0])
            order = np.argsort(h.keys.numpy()[:n])
            assert np.array_equal(h.keys.numpy()[:n][order], exp["keys"])
            assert np.array_equal(h.sums.numpy()[:n][order], exp["sums"])


def test_event_hooks_bracket_the_fused_kernel():
    w = W.config3(2_000_003)
    dims = {d.name: W.device_dim(w, d) for d in w.dims}
    tables = sjq.build_workload_tables(w, dims)
    fact = W.device_fact(w)
    a, b = torch.cuda.Event(enable_timing=True), torch.cuda.Event(enable_timing=True)
    a.record()
    b.record()
    sjq.run_workload(w, fact, tables, sjq.RunOpts(events=(a, b)))
    torch.cuda.synchronize()
    assert 0.0 < a.elapsed_time(b) < 1000.0


def test_prepared_builders_rebuild_identical_tables():
    w = W.config3(400_003)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, tables = run_both(w, fact, hd)
    builders = sjq.workload_builders(w, {k: to_dev(v) for k, v in hd.items()})
    dev_fact = to_dev(fact)
    for _ in range(3):  # rebuilding into the same memory, back to back with runs
        tabs = sjq.build_tables(builders)
        r = sjq.run_workload(w, dev_fact, tabs)
    torch.cuda.synchronize()
    assert all(t.status() == 0 for t in tabs.values())
    for k in tabs:
        assert tabs[k].layout.entries == tables[k].layout.entries and tabs[k].layout.kind == tables[k].layout.kind
    compare(w, r, exp)


def test_open_addressing_tables_give_the_same_result():
    for w in (W.config3(1_200_007), W.config2(900_001)):
        fact = W.host_fact(w)
        hd = {d.name: W.host_dim(w, d) for d in w.dims}
        dev = {k: to_dev(v) for k, v in hd.items()}
        tables = {d.name: sjq.build_dim(dev[d.name], d.key, d.preds, d.payloads, force_kind=sjq.sjq.FORCE_HASH)
                  for d in w.dims}
        assert all(t.layout.kind_name.startswith("HASH") and t.status() == 0 for t in tables.values())
        res, exp, _ = run_both(w, fact, hd, tables=tables)
        assert res.status() == 0
        compare(w, res, exp)
        for opts in (sjq.RunOpts(compaction=1), sjq.RunOpts(compaction=2), sjq.RunOpts(eager_loads=True)):
            res, _, _ = run_both(w, fact, hd, opts=opts, tables=tables)
            compare(w, res, exp)


def test_stale_layout_is_reported_not_followed():
    # plan on one key range, then the data changes before the build: the build must flag it, never write outside
    cols = {"k": torch.arange(1, 1001, dtype=torch.int32, device="cuda"),
            "p": torch.arange(0, 1000, dtype=torch.int32, device="cuda") % 50}
    b = sjq.TableBuilder(cols, "k", (), ("p",))
    b.begin()
    b.scan_side.synchronize()
    cols["k"][7] = 5_000_000       # far outside the planned span
    cols["p"][9] = 100_000         # outside the planned payload range
    t = b.finish()
    torch.cuda.synchronize()
    assert t.status() == 21


def test_reused_layouts_rebuild_without_waiting_and_follow_a_changed_dimension():
    """Builders that reuse the layout of an earlier scan: same tables and result as a planned build while the
    dimension is unchanged; once it changes, the build on the old layout is flagged on the device and a later
    step (the changed statistics have reached the host by then) re-plans and matches the oracle again."""
    for w in (W.config3(400_003), W.config4(300_007, 0.5, 1000, dim_rows=50_000)):
        fact = W.host_fact(w)
        hd = {d.name: W.host_dim(w, d) for d in w.dims}
        _, exp, tables = run_both(w, fact, hd)
        dev_dims = {k: to_dev(v) for k, v in hd.items()}
        builders = sjq.workload_builders(w, dev_dims, reuse_layout=True)
        dev_fact = to_dev(fact)
        for _ in range(4):
            tabs = sjq.build_tables(builders)
            r = sjq.run_workload(w, dev_fact, tabs)
        torch.cuda.synchronize()
        assert all(t.status() == 0 for t in tabs.values())
        for k in tabs:
            assert bytes(tabs[k].layout) == bytes(tables[k].layout)
        compare(w, r, exp)
    # the dimension changes in place: every payload leaves the planned range of its packed code
    hd2 = {"dim": {c: v.copy() for c, v in hd["dim"].items()}}
    hd2["dim"]["w"] += 1000
    dev_dims["dim"]["w"].copy_(torch.from_numpy(hd2["dim"]["w"]))
    torch.cuda.synchronize()
    _, exp2 = oracle_result(w, fact, hd2)
    tabs = sjq.build_tables(builders)  # this step's scan is not waited for: the old layout is used
    torch.cuda.synchronize()
    assert tabs["dim"].status() in (0, 21)  # 21 unless the scan happened to finish before the layout was chosen
    builders["dim"].status.zero_()
    for _ in range(2):
        tabs = sjq.build_tables(builders)
        torch.cuda.synchronize()
    assert tabs["dim"].status() == 0
    assert tabs["dim"].layout.pay_min[0] == tables["dim"].layout.pay_min[0] + 1000
    r = sjq.run_workload(w, dev_fact, tabs)
    torch.cuda.synchronize()
    compare(w, r, exp2)


def test_city_pair_shape_many_groups_few_survivors():
    # two gathered payloads plus the year as group key, 437,500 dense groups, global group table
    w = W.city_pair(3_000_017)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, tables = run_both(w, fact, hd)
    assert res.status() == 0 and res.info.describe()["agg_path"] == "global"
    compare(w, res, exp)
    assert int(res.counts.sum().item()) > 1000
    # the same query with a hashed result list
    wh = replace(w, mode="HASHED", capacity=1 << 16)
    res, exp, _ = run_both(wh, fact, hd, tables=tables)
    assert res.status() == 0
    compare(wh, res, exp)


def test_city_brand_shape_and_the_library_chosen_group_table():
    """The paper's city x brand shape (Section 3.3): year, supplier city and part brand as group key, 1.75 M
    possible groups, about one row in eleven thousand survives.  Asked for as a hashed list, the library picks
    the form of its group table: every term of the key is a gathered payload, so the tables' payload ranges
    bound the key (260,000 cells here); with room for that many cells the table is indexed by the key itself,
    otherwise it is the hash table.  As a dense array of all possible groups it takes global atomics.  All
    three give the oracle's groups bit for bit, with both kernels."""
    w = W.city_brand(6_000_011)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    dev_fact = to_dev(fact)
    tables = None
    for variant, want in ((w, "hash"), (replace(w, capacity=200_000), "global"),
                          (W.city_brand(w.n_rows, hashed=False), "global")):
        for specialise in (False, True):
            res, exp, tables = run_both(variant, fact, hd, opts=sjq.RunOpts(specialise=specialise), dev_fact=dev_fact,
                                        tables=tables)
            assert res.status() == 0 and res.info.describe()["agg_path"] == want
            compare(variant, res, exp)
    assert 300 < exp["counts"].sum() < 900 and tables["supplier"].layout.pay_min[0] == 70
    # the caller can still insist on the hash table
    res, exp, _ = run_both(replace(w, capacity=200_000), fact, hd, opts=sjq.RunOpts(group_hash_always=True),
                           dev_fact=dev_fact, tables=tables)
    assert res.info.describe()["agg_path"] == "hash"
    compare(w, res, exp)


def test_host_path_reads_sparse_columns_in_place_and_matches_copies():
    """sjq_run_host leaves a column that few rows reach in page-locked host memory and lets the kernel read
    it there; copying everything (host_copy_all), pageable buffers (always copied) and the device-resident
    run must all give the oracle's bits.  The transfer plan names what happens to each column."""
    w = W.config3(700_003)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    exp = oracle.run(w, fact, oracle.build_dims(w, hd))
    tables = sjq.build_workload_tables(w, {k: to_dev(v) for k, v in hd.items()})
    pinned = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in fact.items()}
    pinned["unused"] = torch.zeros(w.n_rows, dtype=torch.int32).pin_memory()  # not referenced by the query
    pageable = {k: torch.from_numpy(np.ascontiguousarray(v)) for k, v in fact.items()}
    joins = [(fk, tables[dn]) for fk, dn in w.joins]
    plan = sjq.host_transfer_plan(pinned, w.preds, joins, w.key, w.agg)
    assert plan["suppkey"][0] == "copy" and plan["orderdate"][0] == "copy"
    assert plan["revenue"][0] == "in place" and plan["supplycost"][0] == "in place"
    assert plan["unused"] == ("not transferred", 0.0)
    assert all(how == "copy" or name == "unused" for name, (how, _) in
               sjq.host_transfer_plan(pinned, w.preds, joins, w.key, w.agg, sjq.RunOpts(host_copy_all=True)).items())
    chunk = 131072
    for cols, opts in ((pinned, None), (pinned, sjq.RunOpts(host_copy_all=True)), (pageable, None),
                       (pinned, sjq.RunOpts(specialise=True))):
        staging = torch.empty(sjq.staging_bytes(cols, chunk), dtype=torch.uint8, device="cuda:0")
        res, host = sjq.run_host(cols, staging, chunk, w.preds, joins, w.key, w.agg, w.mode, w.num_groups,
                                 w.capacity, opts)
        torch.cuda.synchronize()
        assert int(host.status[0]) == 0
        assert np.array_equal(host.sums.numpy(), exp["sums"]) and np.array_equal(host.counts.numpy(), exp["counts"])


def test_rows_per_lane_eight_needs_the_specialised_kernel():
    w, fact, hd, _ = ex1()
    tables = sjq.build_workload_tables(w, {k: to_dev(v) for k, v in hd.items()})
    with pytest.raises(sjq.SjqError) as e:
        sjq.run_workload(w, to_dev(fact), tables, sjq.RunOpts(rows_per_lane=8))
    assert e.value.status == 1
    with pytest.raises(sjq.SjqError):
        sjq.run_workload(w, to_dev(fact), tables, sjq.RunOpts(rows_per_lane=5, specialise=True))


def test_hashed_result_with_a_modulo_key_uses_a_direct_table_when_it_fits():
    """Keys taken modulo M lie in (-M, M): with room for 2M - 1 cells the group table is indexed by the key
    (negative keys included), otherwise and on request the hash table is used; same list either way."""
    rng = np.random.default_rng(77)
    n = 50_000
    fact = {"a": rng.integers(-500, 500, n).astype(np.int32), "v": rng.integers(-1000, 1000, n).astype(np.int32)}
    from qhelpers import adhoc
    for modulo, capacity, expect in ((37, 200, "direct"), (37, 20, "hash"), (1, 8, "direct"), (0, 2000, "hash")):
        w = adhoc("modkey", fact, [], [], [Pred("v", "NE", 0)], KeyExpr((Term("FACT", "a", 0, 3),), offset=-7, modulo=modulo),
                  AggExpr("COL", Term("FACT", "v")), "HASHED", capacity=capacity)
        exp = oracle.run(w, fact, oracle.build_dims(w, {}), check=False)
        for opts in (sjq.RunOpts(), sjq.RunOpts(specialise=True), sjq.RunOpts(group_hash_always=True)):
            res = sjq.run_workload(w, to_dev(fact), {}, opts)
            torch.cuda.synchronize()
            if len(exp["keys"]) > capacity:
                assert res.status() == 19
                continue
            assert res.status() == 0
            compare(w, res, exp)
            path = res.info.describe()["agg_path"]
            if expect == "direct" and not opts.group_hash_always:
                assert path in ("global", "shared")
            else:
                assert path == "hash"


@pytest.mark.parametrize("groups", [1000, 100000])
def test_hashed_accumulate_and_host_path_equal_whole(groups):
    """A hashed result accumulated over two calls, and over the chunks of the host-buffer entry point, equals the
    single run (both forms of the group table: indexed by the modulo key, and the hash table)."""
    w = W.config4(400_003, 0.5, groups, hashed=True, dim_rows=50000)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    for opts_kw in ({}, {"group_hash_always": True}, {"specialise": True}):
        res, exp, tables = run_both(w, fact, hd, opts=sjq.RunOpts(**opts_kw))
        compare(w, res, exp)
        k = 150_001
        a = to_dev({c: v[:k] for c, v in fact.items()})
        b = to_dev({c: v[k:].copy() for c, v in fact.items()})
        r = sjq.run_workload(replace(w, n_rows=k), a, tables, sjq.RunOpts(**opts_kw))
        r = sjq.run_workload(replace(w, n_rows=w.n_rows - k), b, tables, sjq.RunOpts(accumulate=True, **opts_kw), result=r)
        torch.cuda.synchronize()
        compare(w, r, exp)
        pinned = {c: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for c, v in fact.items()}
        chunk = 65536
        staging = torch.empty(sjq.staging_bytes(pinned, chunk), dtype=torch.uint8, device="cuda:0")
        rh, host = sjq.run_workload_host(w, pinned, tables, staging, chunk, sjq.RunOpts(**opts_kw))
        torch.cuda.synchronize()
        assert int(host.status[0]) == 0
        compare(w, rh, exp)


def test_key_modulo_one_ignores_its_terms():
    """x % 1 is 0 for every x: the key's columns are not read, the result is the one group 0 (dense or hashed),
    and a column that only the key names is not transferred by the host path."""
    from qhelpers import adhoc
    rng = np.random.default_rng(5)
    n = 30_000
    fact = {"g": rng.integers(-(1 << 30), 1 << 30, n).astype(np.int32), "v": rng.integers(-50, 50, n).astype(np.int32)}
    for mode, kw in (("DENSE", dict(num_groups=1)), ("HASHED", dict(capacity=4))):
        w = adhoc("mod1", fact, [], [], [Pred("v", "GT", -40)], KeyExpr((Term("FACT", "g"),), offset=5, modulo=1),
                  AggExpr("COL", Term("FACT", "v")), mode, **kw)
        exp = oracle.run(w, fact, oracle.build_dims(w, {}))
        for opts in (sjq.RunOpts(), sjq.RunOpts(specialise=True)):
            res = sjq.run_workload(w, to_dev(fact), {}, opts)
            torch.cuda.synchronize()
            assert res.status() == 0
            compare(w, res, exp)
        pinned = {k: torch.from_numpy(v).pin_memory() for k, v in fact.items()}
        plan = sjq.host_transfer_plan(pinned, w.preds, [], w.key, w.agg)
        assert plan["g"][0] == "not transferred" and plan["v"][0] == "copy"


def test_sampled_pass_fractions_track_the_thresholds_of_the_sweep():
    """The planner's selectivity of a fact predicate is measured, not guessed: for the five thresholds of the
    selectivity sweep (0.01 % ... 100 %) the sampled pass fraction is within a factor of two of the true one,
    and planning with it gives the same bits as planning without."""
    n = 40_000_003
    fact = None
    for sel, T in W.C4_THRESHOLDS.items():
        w = W.config4(n, sel, 1000, dim_rows=50_000)
        if fact is None:
            fact = W.device_fact(w)
            tables = sjq.build_workload_tables(w, {d.name: W.device_dim(w, d) for d in w.dims})
        (ppm,) = sjq.sample_preds({"p": fact["p"]}, w.preds)
        assert 0.5 * sel <= ppm / 1e6 <= min(1.0, 2.0 * sel), (sel, ppm)
        a = sjq.run_workload(w, fact, tables)
        b = sjq.run_workload(w, fact, tables, sample=True)
        c = sjq.run_workload(w, fact, tables, sjq.RunOpts(specialise=True, pass_ppm=(ppm,)))
        torch.cuda.synchronize()
        assert a.status() == 0 and b.status() == 0 and c.status() == 0
        assert torch.equal(a.sums, b.sums) and torch.equal(a.counts, b.counts)
        assert torch.equal(a.sums, c.sums) and torch.equal(a.counts, c.counts)
        # exact count of the predicate, from the generator's closed form evaluated with tensor operations
        assert int(a.counts.sum().item()) == int((fact["p"] < T).sum().item())


@pytest.mark.parametrize("seed", range(300, 320))
def test_any_pass_fraction_hint_gives_the_same_result(seed):
    """Hints steer the plan only: right, wrong or extreme measured fractions never change the result."""
    w, fact, hd = random_query(seed, n_fact=900, allow_dup=False, wide_keys=True)
    dev_fact = to_dev(fact)
    tables = None
    nf = len(w.preds) + len(w.joins)
    rng = np.random.default_rng(seed)
    for hints in ((1,) * nf, (1_000_000,) * nf, tuple(int(x) for x in rng.integers(1, 1_000_001, nf))):
        for specialise in (False, True):
            res, exp, tables = run_both(w, fact, hd, opts=sjq.RunOpts(pass_ppm=hints, specialise=specialise),
                                        check=False, dev_fact=dev_fact, tables=tables)
            assert (res.status() == 18) == (exp["status"] == oracle.GROUP_RANGE)
            compare(w, res, exp)


@pytest.mark.parametrize("mk", [lambda: W.config1(1_000_003), lambda: W.config2(2_000_003), lambda: W.config3(2_500_001),
                                lambda: W.config4(1_000_003, 0.5, 1000), lambda: W.config4(1_000_003, 0.1, 100000),
                                lambda: W.config5(1_200_005, 300000), lambda: W.city_brand(3_000_001)])
def test_operator_at_a_time_ablation_matches_the_oracle(mk):
    """The unfused arm of the ablation (one kernel per operator, flag array, materialised payload columns)
    computes the same query: bit-exact against the oracle, and one launch per operator is reported."""
    w = mk()
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    scratch = sjq.unfused_scratch(w.n_rows, len(w.joins))
    res, exp, tables = run_both(w, fact, hd, opts=sjq.RunOpts(unfused_scratch=scratch))
    assert res.status() == 0
    compare(w, res, exp)
    passes = len(w.preds) + sum(2 if (t.layout.kind in (6, 7) and t.layout.filter_bits) else 1 for t in tables.values())
    assert res.info.kernel_launches == 1 + passes + 1 + (1 if w.mode == "HASHED" else 0)
    # too little scratch is refused on the host
    with pytest.raises(sjq.SjqError) as e:
        sjq.run_workload(w, to_dev(fact), tables, sjq.RunOpts(unfused_scratch=scratch[: w.n_rows // 2]))
    assert e.value.status == 5


def _hot_variants():
    return [sjq.RunOpts(hot_keys=1), sjq.RunOpts(hot_keys=1, specialise=True), sjq.RunOpts(hot_keys=2),
            sjq.RunOpts(hot_keys=1, compaction=1), sjq.RunOpts(hot_keys=1, specialise=True, compaction=2),
            sjq.RunOpts(hot_keys=1, eager_loads=True)]


def test_hot_key_table_skewed_keys_against_the_oracle():
    """The hot-key table of an open-addressing join (heaviest foreign keys answered from shared memory): the
    Zipf-skewed 64-bit-key shape, where three quarters of the heavy keys are absent from the filtered dimension,
    bit for bit against the oracle with the table forced on, off, and in every kernel form."""
    w = W.config5(1_300_007, 300_000)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    dev_fact = to_dev(fact)
    tables = None
    for opts in _hot_variants():
        res, exp, tables = run_both(w, fact, hd, opts=opts, dev_fact=dev_fact, tables=tables)
        assert res.status() == 0
        compare(w, res, exp)
    assert int(res.counts.sum().item()) > 100_000
    # the table really was in use: its header (after the count table, the claims and 2048 entries) counts the keys
    # held, and together they cover a good part of the sampled rows
    scratch = torch.empty(sjq.sjq.HOT_SCRATCH_BYTES, dtype=torch.uint8, device="cuda")
    res, exp, _ = run_both(w, fact, hd, opts=sjq.RunOpts(hot_keys=1, hot_scratch=scratch), dev_fact=dev_fact,
                           tables=tables)
    compare(w, res, exp)
    held, _, covered, _ = scratch[(1 << 18) * 12 + 2048 * 4 + 2048 * 16:][:16].view(torch.int32).tolist()
    assert held > 500 and covered > 0.3 * min(w.n_rows, 1 << 18)


def test_hot_key_table_uniform_keys_and_32_bit_keys():
    # four open-addressing joins on 32-bit keys with payload codes (the first one gets the hot table); the keys
    # are uniform, so the table stays empty or thin: either way the result is the oracle's
    w = W.config3(1_200_007)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    dev = {k: to_dev(v) for k, v in hd.items()}
    tables = {d.name: sjq.build_dim(dev[d.name], d.key, d.preds, d.payloads, force_kind=sjq.sjq.FORCE_HASH)
              for d in w.dims}
    dev_fact = to_dev(fact)
    for opts in _hot_variants():
        res, exp, _ = run_both(w, fact, hd, opts=opts, dev_fact=dev_fact, tables=tables)
        assert res.status() == 0
        compare(w, res, exp)


def test_hot_key_table_heavy_keys_with_special_values():
    """A few keys carry nearly all rows, among them -1 (the count table's free-slot pattern), the table's empty
    marker (never a key: always a miss) and keys the dimension does not hold."""
    rng = np.random.default_rng(7)
    n = 400_003
    dim_keys = np.concatenate([np.array([-1, 5, 7_000_000_000, -9_000_000_000], dtype=np.int64),
                               rng.integers(-2**62, 2**62, 5000, dtype=np.int64)])
    dim = {"key": dim_keys, "pay": rng.integers(0, 1000, len(dim_keys)).astype(np.int32),
           "attr": rng.integers(0, 4, len(dim_keys)).astype(np.int32)}
    dim["attr"][:4] = [0, 0, 3, 0]  # 7_000_000_000 is filtered out: a heavy absent key
    heavy = np.array([-1, 5, 7_000_000_000, -9_000_000_000, np.iinfo(np.int64).min, 123456789], dtype=np.int64)
    pick = rng.integers(0, 100, n)
    fk = np.where(pick < 90, heavy[pick % len(heavy)], dim_keys[rng.integers(0, len(dim_keys), n)])
    fact = {"fk": fk.astype(np.int64), "m": rng.integers(0, 1_000_000, n).astype(np.int32)}
    w = adhoc("hot_special", fact, [("dim", dim, "key", [Pred("attr", "LT", 3)], ["pay"], True)], [("fk", "dim")], [],
              KeyExpr((Term("PAYLOAD", 0, 0),), modulo=64), AggExpr("COL", Term("FACT", "m")), "DENSE", num_groups=64)
    tables = None
    for opts in _hot_variants():
        res, exp, tables = run_both(w, fact, {"dim": dim}, opts=opts, tables=tables)
        assert res.status() == 0
        compare(w, res, exp)


def test_wrapping_product_matches_the_oracle():
    # products beyond 63 bits wrap modulo 2^64 the same way on both sides (scalar and grouped)
    rng = np.random.default_rng(11)
    n = 10_007
    fact = {"x": rng.integers(-2**62, 2**62, n, dtype=np.int64), "y": rng.integers(-2**62, 2**62, n, dtype=np.int64),
            "g": rng.integers(0, 50, n).astype(np.int32)}
    agg = AggExpr("MUL", Term("FACT", "x", 0, 3), Term("FACT", "y", 0, -5))
    for w in (adhoc("wrapmul", fact, [], [], [], None, agg, "SCALAR"),
              adhoc("wrapmul_g", fact, [], [], [], KeyExpr((Term("FACT", "g"),)), agg, "DENSE", num_groups=50)):
        for opts in (sjq.RunOpts(), sjq.RunOpts(specialise=True)):
            res, exp, _ = run_both(w, fact, {}, opts=opts)
            assert res.status() == 0
            compare(w, res, exp)


@pytest.mark.parametrize("n,capacity", [(0, 8), (1, 1), (5, 64), (1023, 1024), (1025, 4096), (100_003, 131_072),
                                        (300_000, 300_000)])
def test_result_sort_orders_triples_by_signed_key(n, capacity):
    # distinct keys over the whole signed range, special values included; entries past n_groups stay untouched
    rng = np.random.default_rng(n + 1)
    keys = np.unique(np.concatenate([rng.integers(-2**63, 2**63 - 1, n + 16, dtype=np.int64),
                                     np.array([0, -1, 1, np.iinfo(np.int64).min, np.iinfo(np.int64).max, 255, 256,
                                               -256, 2**32, -2**32], dtype=np.int64)]))
    keys = rng.permutation(keys)[:n]
    sums = rng.integers(-2**62, 2**62, capacity, dtype=np.int64)
    counts = rng.integers(0, 2**40, capacity, dtype=np.int64)
    allk = np.full(capacity, 77, dtype=np.int64)
    allk[:n] = keys
    res = sjq.Result("HASHED", torch.from_numpy(sums.copy()).cuda(), torch.from_numpy(counts.copy()).cuda(),
                     torch.from_numpy(allk.copy()).cuda(), torch.tensor([n], dtype=torch.int64, device="cuda"),
                     torch.zeros(1, dtype=torch.int32, device="cuda"), None)
    res.sort()
    torch.cuda.synchronize()
    order = np.argsort(keys, kind="stable")
    assert np.array_equal(res.keys.cpu().numpy()[:n], keys[order])
    assert np.array_equal(res.sums.cpu().numpy()[:n], sums[:n][order])
    assert np.array_equal(res.counts.cpu().numpy()[:n], counts[:n][order])
    assert np.array_equal(res.keys.cpu().numpy()[n:], allk[n:])
    assert np.array_equal(res.sums.cpu().numpy()[n:], sums[n:])
    assert np.array_equal(res.counts.cpu().numpy()[n:], counts[n:])


def test_open_addressing_table_at_a_16_byte_aligned_address():
    """Table memory only has to be 16-byte aligned; a bucket array that does not start on a 32-byte boundary is
    probed with two 128-bit loads instead of one 256-bit load.  Same result either way."""
    w = W.config5(700_001, 100_000)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    d = w.dims[0]
    dev = to_dev(hd[d.name])
    for off in (0, 16):
        t = sjq.build_dim(dev, d.key, d.preds, d.payloads, force_kind=sjq.sjq.FORCE_HASH, mem_offset=off).check()
        assert t.mem.data_ptr() % 32 == off
        for opts in (sjq.RunOpts(), sjq.RunOpts(specialise=True), sjq.RunOpts(specialise=True, hot_keys=1)):
            res, exp, _ = run_both(w, fact, hd, opts=opts, tables={d.name: t})
            assert res.status() == 0
            compare(w, res, exp)
