"""Parity of the run-time specialised fused kernel (sjq_run_opts.specialise)
with the CPU oracle: the same bits as the interpreted kernel, on the same
seeded inputs, over query shapes, option switches, ragged sizes and edge cases."""
import ctypes

import numpy as np
import pytest
import torch

import oracle
from datagen import workloads as W
from datagen.workloads import AggExpr, KeyExpr, Pred, Term

pytestmark = pytest.mark.gpu

sjq = pytest.importorskip("paper_2607_07632_b200") if torch.cuda.is_available() else None

from gpuhelpers import compare, run_both, to_dev  # noqa: E402
from qhelpers import ex1, ex2, ex3, random_query  # noqa: E402


def spec(**kw):
    return sjq.RunOpts(specialise=True, **kw)


def test_hand_examples_specialised():
    for mk in (ex1, ex2, ex3):
        w, fact, hd, _ = mk()
        res, exp, _ = run_both(w, fact, hd, opts=spec())
        assert res.status() == 0
        compare(w, res, exp)


@pytest.mark.parametrize("seed", range(300, 348))
def test_random_small_queries_specialised(seed):
    w, fact, hd = random_query(seed, allow_dup=False, wide_keys=True)
    res, exp, _ = run_both(w, fact, hd, opts=spec(), check=False)
    assert (res.status() == 18) == (exp["status"] == oracle.GROUP_RANGE)
    compare(w, res, exp)


@pytest.mark.parametrize("seed", range(348, 356))
def test_random_queries_option_matrix_specialised(seed):
    w, fact, hd = random_query(seed, n_fact=700, allow_dup=False, wide_keys=True)
    dev_fact = to_dev(fact)
    tables = None
    for opts in (spec(eager_loads=True), spec(smem_tables=1), spec(block_threads=128, ctas_per_sm=1),
                 spec(block_threads=1024, ctas_per_sm=1), spec(block_threads=512, compaction=2, smem_tables=2),
                 spec(agg_path=2), spec(compaction=1), spec(rows_per_lane=8), spec(rows_per_lane=8, compaction=2),
                 spec(no_filter_bitmap=True), spec(group_hash_always=True), spec(dense_slots=4), spec(dense_slots=4, block_threads=768, ctas_per_sm=1),
                 spec(warp_agg=1), spec(warp_agg=1, agg_path=2), spec(warp_agg=2, compaction=1),
                 spec(hot_keys=1), spec(hot_keys=1, l0_bulk=1, block_threads=256, ctas_per_sm=2), spec(l0_bulk=1, compaction=2),
                 spec(pass_ppm=(900_000,) * (len(w.preds) + len(w.joins))),  # "most rows survive": the queue-free plan
                 spec(order=tuple(reversed(range(len(w.preds) + len(w.joins)))))):
        res, exp, tables = run_both(w, fact, hd, opts=opts, check=False, dev_fact=dev_fact, tables=tables)
        assert (res.status() == 18) == (exp["status"] == oracle.GROUP_RANGE)
        compare(w, res, exp)


@pytest.mark.parametrize("n", [0, 1, 5, 257, 3071, 3073, 100003])
@pytest.mark.parametrize("cfg", ["c1", "c2", "c3", "c4d", "c4h", "c5"])
def test_configs_ragged_sizes_specialised(cfg, n):
    w = {"c1": lambda: W.config1(n), "c2": lambda: W.config2(n), "c3": lambda: W.config3(n),
         "c4d": lambda: W.config4(n, 0.5, 1000, dim_rows=50000),
         "c4h": lambda: W.config4(n, 0.5, 100000, dim_rows=50000),
         "c5": lambda: W.config5(n, 20000)}[cfg]()
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, _ = run_both(w, fact, hd, opts=spec())
    assert res.status() == 0
    compare(w, res, exp)


@pytest.mark.parametrize("mk", [lambda: W.config1(1_500_007), lambda: W.config2(2_000_003),
                                lambda: W.config3(2_500_001), lambda: W.config5(1_200_005, 300000),
                                lambda: W.city_pair(1_000_003)] +
                         [lambda s=s, g=g: W.config4(1_000_003, s, g) for s in (0.0001, 0.1, 1.0)
                          for g in (1, 1000, 100000, 1000000)])
def test_configs_multi_tile_specialised(mk):
    w = mk()
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, tables = run_both(w, fact, hd, opts=spec())
    assert res.status() == 0
    compare(w, res, exp)
    dev_fact = to_dev(fact)
    nf = len(w.preds) + len(w.joins)
    for opts in (spec(eager_loads=True, smem_tables=1, compaction=1),
                 spec(agg_path=2 if w.mode == "DENSE" else 0, block_threads=768, ctas_per_sm=1, compaction=2),
                 spec(rows_per_lane=8, no_filter_bitmap=True, smem_tables=2), spec(dense_slots=4),
                 spec(warp_agg=1), spec(warp_agg=1, agg_path=1 if (w.mode == "DENSE" and 1 < w.num_groups <= 4096) else 0),
                 spec(pass_ppm=(950_000,) * nf), spec(pass_ppm=(950_000,) * nf, warp_agg=1, block_threads=256)):
        res2, _, _ = run_both(w, fact, hd, opts=opts, dev_fact=dev_fact, tables=tables)
        compare(w, res2, exp)


def test_one_module_serves_runs_that_differ_only_in_data_dependent_values():
    """Thresholds, key ranges and table contents are kernel parameters, not part of the compiled shape:
    changing them must not need (or wrongly reuse state of) another module, and the results stay exact."""
    n = 200_003
    for t in (1, 100, 5000, 10000):
        w = W.config4(n, t / 10000.0, 1000, dim_rows=30000 + t)
        fact = W.host_fact(w)
        hd = {d.name: W.host_dim(w, d) for d in w.dims}
        res, exp, _ = run_both(w, fact, hd, opts=spec())
        assert res.status() == 0
        compare(w, res, exp)


def test_group_range_and_overflow_status_specialised():
    w, fact, hd, _ = ex2()
    from dataclasses import replace
    small = replace(w, num_groups=1500)  # keys 2020 fall outside
    res, exp, _ = run_both(small, fact, hd, opts=spec(), check=False)
    assert res.status() == 18 and exp["status"] == oracle.GROUP_RANGE
    compare(small, res, exp)


def test_host_buffer_entry_point_specialised():
    w = W.config3(300_007)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    dims = oracle.build_dims(w, hd)
    exp = oracle.run(w, fact, dims)
    tables = sjq.build_workload_tables(w, {k: to_dev(v) for k, v in hd.items()})
    host_fact = {k: torch.from_numpy(np.ascontiguousarray(v)).pin_memory() for k, v in fact.items()}
    chunk = 65536
    staging = torch.empty(sjq.staging_bytes(host_fact, chunk), dtype=torch.uint8, device="cuda:0")
    res, host = sjq.run_workload_host(w, host_fact, tables, staging, chunk, spec())
    torch.cuda.synchronize()
    assert np.array_equal(host.sums.numpy(), exp["sums"])


def test_compiler_log_is_readable():
    L = sjq.sjq.lib()
    L.sjq_jit_log.restype = ctypes.c_size_t
    L.sjq_jit_log.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
    buf = ctypes.create_string_buffer(4096)
    n = L.sjq_jit_log(buf, len(buf))
    assert n >= 0 and len(buf.value) <= 4095


@pytest.mark.parametrize("seed", [900, 901, 902])
def test_largest_query_shape_both_kernels(seed):
    """Sixteen predicates and eight joins (the limits of the interface), several with two payloads: the
    interpreted kernel walks about forty stage descriptors, the specialised one unrolls them all."""
    from dataclasses import replace

    w, fact, hd = random_query(seed, n_fact=600, n_joins=8, allow_dup=False, wide_keys=True)
    rng = np.random.default_rng(seed)
    preds = []
    for i in range(16):
        col = f"c{i % 3}"
        kind = i % 4
        if kind == 0:
            preds.append(Pred(col, "BETWEEN", -4, int(rng.integers(8, 12))))
        elif kind == 1:
            preds.append(Pred(col, "NE", int(rng.integers(-4, 12))))
        elif kind == 2:
            preds.append(Pred(col, "GE", int(rng.integers(-4, -1))))
        else:
            preds.append(Pred(col, "IN", values=tuple(range(-4, int(rng.integers(6, 12))))))
    w = replace(w, preds=tuple(preds))
    dev_fact = to_dev(fact)
    tables = None
    for opts in (sjq.RunOpts(), spec(), spec(compaction=1)):
        res, exp, tables = run_both(w, fact, hd, opts=opts, check=False, dev_fact=dev_fact, tables=tables)
        assert (res.status() == 18) == (exp["status"] == oracle.GROUP_RANGE)
        compare(w, res, exp)


@pytest.mark.parametrize("seed", range(400, 430))
def test_random_queries_over_many_tiles_both_kernels(seed):
    """Random query shapes over a fact table of several tiles with a ragged tail (the hand-sized random
    queries fit one tile): queues fill, drain and wrap for shapes no configuration has."""
    n = 20_000 + 37 * (seed % 7) + (seed % 4)
    w, fact, hd = random_query(seed, n_fact=n, max_dim=40, allow_dup=False, wide_keys=True)
    dev_fact = to_dev(fact)
    tables = None
    for opts in (sjq.RunOpts(), spec(), spec(block_threads=128, ctas_per_sm=4), sjq.RunOpts(compaction=2)):
        res, exp, tables = run_both(w, fact, hd, opts=opts, check=False, dev_fact=dev_fact, tables=tables)
        assert (res.status() == 18) == (exp["status"] == oracle.GROUP_RANGE)
        compare(w, res, exp)


def test_clearing_the_module_cache_recompiles_and_gives_the_same_bits():
    w, fact, hd, _ = ex2()
    res, exp, tables = run_both(w, fact, hd, opts=spec())
    compare(w, res, exp)
    torch.cuda.synchronize()
    L = sjq.sjq.lib()
    L.sjq_jit_cache_clear.restype = ctypes.c_int32
    assert L.sjq_jit_cache_clear() >= 1
    assert L.sjq_jit_cache_clear() == 0
    res2, _, _ = run_both(w, fact, hd, opts=spec(), tables=tables)
    compare(w, res2, exp)


BULK_SHAPES = [dict(), dict(block_threads=1024, ctas_per_sm=1), dict(dense_slots=4),
               dict(block_threads=128, ctas_per_sm=2, compaction=2), dict(rows_per_lane=8)]


@pytest.mark.parametrize("n", [0, 1, 255, 3071, 3072, 3073, 6145, 100003, 1_200_011])
@pytest.mark.parametrize("cfg", ["c1", "c3", "c4d", "c4h", "c5"])
def test_first_column_staged_by_bulk_copies(cfg, n):
    """The first column brought into shared memory by bulk-asynchronous copies (one slice per warp and tile,
    completion on an mbarrier with a bounded wait): int32 and int64 first columns, whole tiles, ragged tails
    and tables smaller than one tile, several block shapes; bit for bit against the oracle, and the bounded
    waits never ran out (status 0)."""
    w = {"c1": lambda: W.config1(n), "c3": lambda: W.config3(n),
         "c4d": lambda: W.config4(n, 0.1, 1000, dim_rows=50000), "c4h": lambda: W.config4(n, 0.01, 100000, dim_rows=50000),
         "c5": lambda: W.config5(n, 20000)}[cfg]()
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    dev_fact = to_dev(fact)
    tables = None
    for shape in BULK_SHAPES if n > 3000 else BULK_SHAPES[:2]:
        res, exp, tables = run_both(w, fact, hd, opts=spec(l0_bulk=1, **shape), dev_fact=dev_fact, tables=tables)
        assert res.status() == 0
        compare(w, res, exp)


@pytest.mark.parametrize("seed", range(360, 372))
def test_random_queries_with_bulk_staging(seed):
    w, fact, hd = random_query(seed, n_fact=9000, allow_dup=False, wide_keys=True)
    res, exp, _ = run_both(w, fact, hd, opts=spec(l0_bulk=1, block_threads=128, ctas_per_sm=1), check=False)
    assert (res.status() == 18) == (exp["status"] == oracle.GROUP_RANGE)
    compare(w, res, exp)


def test_bulk_copy_wait_that_runs_out_is_reported_and_survived():
    """The failure path of the bulk-asynchronous staging, reached without faulting anything: the kernel waits
    for copies that are never issued, every bounded wait runs out, the status word says so and the kernel
    finishes the query with plain loads: same bits as the oracle."""
    w = W.config4(20_011, 0.5, 1000, dim_rows=50000)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    res, exp, tables = run_both(w, fact, hd, opts=spec(l0_bulk=3, block_threads=128, ctas_per_sm=1, compaction=2))
    assert res.status() == 22
    compare(w, res, exp)
    # the context is still usable and the same query without the switch is clean
    res, exp, _ = run_both(w, fact, hd, opts=spec(l0_bulk=1, block_threads=128, ctas_per_sm=1, compaction=2), tables=tables)
    assert res.status() == 0
    compare(w, res, exp)
