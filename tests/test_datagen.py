"""The synthetic-input definition: calendar pins, ranges, determinism."""
import numpy as np

import datagen
from datagen import workloads as W


def test_calendar_pins():
    w = W.config1(10)
    d = W.host_dim(w, w.dims[0])
    assert d["datekey"].size == 2556
    assert d["datekey"][0] == 19920101 and d["datekey"][-1] == 19981230
    assert (d["year"] == 1992).sum() == 366 and (d["year"] == 1993).sum() == 365
    assert (d["year"] == 1996).sum() == 366 and (d["year"] == 1998).sum() == 364
    assert 19920229 in d["datekey"] and 19930229 not in d["datekey"]
    assert d["datekey"].max() - d["datekey"].min() + 1 == 61130
    assert np.array_equal(d["year"], d["datekey"] // 10000)
    assert np.all(np.diff(d["datekey"]) > 0)


def test_uniform_ranges_inclusive():
    w = W.config1(300000)
    f = W.host_fact(w)
    assert (f["discount"].min(), f["discount"].max()) == (0, 10)
    assert (f["quantity"].min(), f["quantity"].max()) == (1, 50)
    assert f["extendedprice"].min() >= 90000 and f["extendedprice"].max() <= 10000000
    assert np.bincount(f["discount"]).min() > 300000 / 11 * 0.95


def test_pure_function_of_row():
    w = W.config3(5000)
    whole = W.host_fact(w)
    part = W.host_fact(w, 1234, 1000)
    for k in whole:
        assert np.array_equal(whole[k][1234:2234], part[k])


def test_region_is_nation_div_5():
    w = W.config3(10)
    c = W.host_dim(w, w.dim("customer"))
    assert np.array_equal(c["region"], c["nation"] // 5)
    assert np.array_equal(c["custkey"], np.arange(1, 3000001, dtype=np.int32))


def test_mix_is_injective_on_a_range_and_zipf_shape():
    w = W.config5(200000, 10000)
    d = W.host_dim(w, w.dims[0])
    assert np.unique(d["key"]).size == 10000
    f = W.host_fact(w)
    assert np.isin(f["fk"], d["key"]).all()
    # rank-1 share ~ 1/H_K
    H = (1.0 / np.arange(1, 10001)).sum()
    share = (f["fk"] == d["key"][0]).mean()
    assert abs(share - 1 / H) < 0.01
    cum = datagen.zipf_table(10000)
    assert cum[0] == 1 << 40 and cum[1] - cum[0] == (1 << 40) // 2 and np.all(np.diff(cum.astype(np.int64)) > 0)
