"""Pins for the CPU oracle: every check compares it with something other than
itself -- hand-computed examples, brute-force nested loops, closed forms and
invariants of the query definition."""
import numpy as np
import pytest
from dataclasses import replace

import oracle
from datagen import workloads as W
from datagen.workloads import AggExpr, KeyExpr, Pred, Term

from bruteforce import brute, dup_keys_among_passing
from qhelpers import adhoc, ex1, ex2, ex3, random_query


def _run(w, fact, host_dims, **kw):
    dims = oracle.build_dims(w, host_dims)
    return oracle.run(w, fact, dims, **kw)


def test_hand_example_1_scalar():
    w, fact, hd, exp = ex1()
    r = _run(w, fact, hd)
    assert (r["sum"], r["count"]) == (exp["sum"], exp["count"]) == (41980000, 4)


def test_hand_example_2_groupby():
    w, fact, hd, exp = ex2()
    r = _run(w, fact, hd)
    nz = {int(k): [int(r["sums"][k]), int(r["counts"][k])] for k in np.nonzero(r["counts"])[0]}
    assert nz == exp
    assert int(r["sums"].sum()) == 1500


def test_hand_example_3_int64_hashed_truncating_mod():
    w, fact, hd, exp = ex3()
    r = _run(w, fact, hd)
    got = {int(k): [int(s), int(c)] for k, s, c in zip(r["keys"], r["sums"], r["counts"])}
    assert got == exp
    assert list(r["keys"]) == sorted(r["keys"])  # canonical ascending order


@pytest.mark.parametrize("seed", range(300))
def test_brute_force_random_queries(seed):
    w, fact, hd = random_query(seed, allow_dup=True, wide_keys=True)
    kind, groups, oor = brute(w, fact, hd)
    dims = oracle.build_dims(w, hd)
    dup = any(dup_keys_among_passing(w.dim(dn), hd[dn]) for _, dn in w.joins)
    assert dup == any(d.status == oracle.DUP_KEY for d in dims.values())
    if dup:
        return
    r = oracle.run(w, fact, dims, check=False)
    assert (r["status"] == oracle.GROUP_RANGE) == oor
    if w.mode == "SCALAR":
        s, c = groups.get(0, [0, 0])
        assert (r["sum"], r["count"]) == (s, c)
    elif w.mode == "DENSE":
        exp_s = np.zeros(w.num_groups, np.int64)
        exp_c = np.zeros(w.num_groups, np.int64)
        for k, (s, c) in groups.items():
            exp_s[k], exp_c[k] = s, c
        assert np.array_equal(r["sums"], exp_s) and np.array_equal(r["counts"], exp_c)
    else:
        ks = sorted(groups)
        assert list(r["keys"]) == ks
        assert [int(x) for x in r["sums"]] == [groups[k][0] for k in ks]
        assert [int(x) for x in r["counts"]] == [groups[k][1] for k in ks]


def test_closed_form_plain_sum_and_count():
    # no predicates, no joins, scalar: the query is sum(col) and count = N
    w = W.config1(100003)
    fact = W.host_fact(w)
    q = replace(w, joins=(), dims=(), preds=(), agg=AggExpr("COL", Term("FACT", "extendedprice")))
    r = _run(q, fact, {})
    assert r["sum"] == int(fact["extendedprice"].astype(np.int64).sum()) and r["count"] == 100003


def test_closed_form_numpy_mask_c1():
    # the whole of config 1 restated with boolean masks and np.isin
    w = W.config1(200001)
    fact = W.host_fact(w)
    hd = {"date": W.host_dim(w, w.dims[0])}
    keep = hd["date"]["datekey"][hd["date"]["year"] == 1993]
    m = (np.isin(fact["orderdate"], keep) & (fact["discount"] >= 2) & (fact["discount"] <= 4)
         & (fact["quantity"] < 30))
    exp = int((fact["extendedprice"][m].astype(np.int64) * fact["discount"][m]).sum())
    r = _run(w, fact, hd)
    assert (r["sum"], r["count"]) == (exp, int(m.sum()))


def test_closed_form_numpy_c3_groupby():
    w = W.config3(300007)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    c, s, p, d = hd["customer"], hd["supplier"], hd["part"], hd["date"]
    nation = c["nation"][fact["custkey"] - 1]
    year = np.zeros(20000000, np.int32)
    year[d["datekey"]] = d["year"]
    yr = year[fact["orderdate"]]
    m = ((c["region"][fact["custkey"] - 1] == 1) & (s["region"][fact["suppkey"] - 1] == 1)
         & (p["mfgr"][fact["partkey"] - 1] <= 1) & (yr >= 1997) & (yr <= 1998))
    g = (yr[m] - 1992) * 25 + nation[m]
    v = fact["revenue"][m].astype(np.int64) - fact["supplycost"][m]
    exp_s = np.bincount(g, weights=None, minlength=175) * 0
    exp_s = np.zeros(175, np.int64)
    np.add.at(exp_s, g, v)
    exp_c = np.bincount(g, minlength=175)
    r = _run(w, fact, hd)
    assert np.array_equal(r["sums"], exp_s) and np.array_equal(r["counts"], exp_c)
    assert np.count_nonzero(r["counts"]) == 10  # 2 years x 5 nations of region 1


def test_c4_count_is_threshold_count():
    for sel, T in W.C4_THRESHOLDS.items():
        w = W.config4(50000, sel, 1000, dim_rows=5000)
        fact = W.host_fact(w)
        hd = {"dim": W.host_dim(w, w.dims[0])}
        r = _run(w, fact, hd)
        m = fact["p"] < T
        assert int(r["counts"].sum()) == int(m.sum())
        exp = int(fact["m"][m].astype(np.int64).sum() + hd["dim"]["w"][fact["fk"][m] - 1].astype(np.int64).sum())
        assert int(r["sums"].sum()) == exp


def test_empty_cases():
    w = W.config2(5000)
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    # dimension filter keeping nothing -> every probe misses
    d0 = replace(w.dims[1], preds=(Pred("region", "EQ", 99),))
    q = replace(w, dims=(w.dims[0], d0, w.dims[2]))
    r = _run(q, fact, hd)
    assert r["sums"].sum() == 0 and r["counts"].sum() == 0
    # zero fact rows
    r = _run(w, {k: v[:0] for k, v in fact.items()}, hd)
    assert r["counts"].sum() == 0


def _groups(r, w):
    if w.mode == "SCALAR":
        return {0: (r["sum"], r["count"])} if r["count"] else {}
    if w.mode == "DENSE":
        return {int(k): (int(r["sums"][k]), int(r["counts"][k])) for k in np.nonzero(r["counts"])[0]}
    return {int(k): (int(s), int(c)) for k, s, c in zip(r["keys"], r["sums"], r["counts"])}


@pytest.mark.parametrize("mk", [lambda: W.config1(40001), lambda: W.config2(60001), lambda: W.config3(80001),
                                lambda: W.config4(30001, 0.5, 1000, dim_rows=4000),
                                lambda: W.config4(30001, 0.5, 100000, dim_rows=4000),
                                lambda: W.config5(30001, 5000)])
def test_invariants(mk):
    w = mk()
    fact = W.host_fact(w)
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    dims = oracle.build_dims(w, hd)
    whole = oracle.run(w, fact, dims)
    G = _groups(whole, w)
    rng = np.random.default_rng(7)
    # split-and-add at an arbitrary row
    k = 12345
    a = _groups(oracle.run(w, fact, dims, 0, k), w)
    b = _groups(oracle.run(w, fact, dims, k, w.n_rows), w)
    merged = {}
    for part in (a, b):
        for key, (s, c) in part.items():
            s0, c0 = merged.get(key, (0, 0))
            merged[key] = (s0 + s, c0 + c)
    assert merged == G
    # permutation of fact rows
    perm = rng.permutation(w.n_rows)
    assert _groups(oracle.run(w, {n: v[perm] for n, v in fact.items()}, dims), w) == G
    # permutation of dimension rows
    hd2 = {}
    for d in w.dims:
        p = rng.permutation(d.rows)
        hd2[d.name] = {n: v[p] for n, v in hd[d.name].items()}
    assert _groups(oracle.run(w, fact, oracle.build_dims(w, hd2)), w) == G
    # join order and predicate order (payload indices of key terms follow the joins)
    if len(w.joins) > 1:
        order = list(range(len(w.joins)))[::-1]
        inv = {old: new for new, old in enumerate(order)}

        def remap(t):
            return replace(t, a=inv[t.a]) if t is not None and t.src == "PAYLOAD" else t

        key = replace(w.key, terms=tuple(remap(t) for t in w.key.terms)) if w.key else None
        agg = replace(w.agg, x=remap(w.agg.x), y=remap(w.agg.y))
        q = replace(w, joins=tuple(w.joins[i] for i in order), preds=w.preds[::-1], key=key, agg=agg)
        assert _groups(oracle.run(q, fact, dims), w) == G
    # sum over groups equals the scalar query with the same filters
    sc = oracle.run(replace(w, mode="SCALAR", key=None), fact, dims)
    assert sum(s for s, _ in G.values()) == sc["sum"] and sum(c for _, c in G.values()) == sc["count"]


def test_unused_unfiltered_dimension_changes_nothing():
    w = W.config4(20001, 0.5, 1000, dim_rows=3000)
    fact = W.host_fact(w)
    hd = {"dim": W.host_dim(w, w.dims[0])}
    base = _run(w, fact, hd)
    q = replace(w, joins=(), dims=(), agg=AggExpr("COL", Term("FACT", "m")))
    nojoin = _run(q, fact, {})
    assert np.array_equal(base["counts"], nojoin["counts"])  # every fk hits the unfiltered dimension


def test_statistics_of_configs():
    # survivors within 5 sigma of N * product of selectivities (sanity, not parity)
    for w, p in ((W.config1(400000), 365 / 2556 * 3 / 11 * 29 / 50), (W.config2(400000), 1 / 25 / 5),
                 (W.config3(400000), 1 / 5 * 1 / 5 * 2 / 5 * 729 / 2556)):
        fact = W.host_fact(w)
        hd = {d.name: W.host_dim(w, d) for d in w.dims}
        r = _run(w, fact, hd)
        cnt = r["count"] if w.mode == "SCALAR" else int(r["counts"].sum())
        # dimension filters are themselves random draws, so allow a generous band
        assert abs(cnt - w.n_rows * p) < 0.12 * w.n_rows * p + 5 * np.sqrt(w.n_rows * p)


def test_missing_and_out_of_range_fk_is_a_miss():
    fact = {"fk": np.array([-7, 0, 1, 5, 6, 2**31 - 1, -2**31], np.int32), "v": np.arange(7, dtype=np.int32) + 1}
    dim = {"k": np.array([1, 5], np.int32), "p": np.array([3, 4], np.int32)}
    w = adhoc("miss", fact, [("d", dim, "k", [], ["p"])], [("fk", "d")], [], None,
              AggExpr("MUL", Term("FACT", "v"), Term("PAYLOAD", 0, 0)), "SCALAR")
    r = _run(w, fact, {"d": dim})
    assert (r["sum"], r["count"]) == (3 * 3 + 4 * 4, 2)


def test_dense_group_range_flag():
    fact = {"g": np.array([0, 3, 4, -1], np.int32)}
    w = adhoc("range", fact, [], [], [], KeyExpr((Term("FACT", "g"),)), AggExpr("COL", Term("FACT", "g")), "DENSE",
              num_groups=4)
    r = oracle.run(w, fact, {}, check=False)
    assert r["status"] == oracle.GROUP_RANGE
    assert list(r["counts"]) == [1, 0, 0, 1]


def test_sum_wraps_modulo_2_64():
    fact = {"v": np.array([2**62, 2**62, 2**62, 2**62, 5], np.int64)}
    w = adhoc("wrap", fact, [], [], [], None, AggExpr("COL", Term("FACT", "v")), "SCALAR")
    assert _run(w, fact, {})["sum"] == 5


def _wrap64(x: int) -> int:
    x &= (1 << 64) - 1
    return x - (1 << 64) if x >= (1 << 63) else x


def test_product_wraps_modulo_2_64():
    # x * y beyond 63 bits, scaled terms included: the sum is the exact integer result reduced modulo 2^64
    x = np.array([2**40, -(2**45), 3037000500, 2**62, -7], np.int64)
    y = np.array([2**30, 2**33, 3037000500, 6, 2**61], np.int64)
    fact = {"x": x, "y": y}
    w = adhoc("wrapmul", fact, [], [], [], None, AggExpr("MUL", Term("FACT", "x", 0, 3), Term("FACT", "y", 0, -5)), "SCALAR")
    exact = sum(int(a) * 3 * int(b) * -5 for a, b in zip(x, y))
    assert exact.bit_length() > 64
    assert _run(w, fact, {})["sum"] == _wrap64(exact)
