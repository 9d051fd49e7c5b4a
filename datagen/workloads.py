"""Plain-data descriptions of the five benchmark workloads and of small test
queries: which columns exist (and how the generator fills them) and what the
query asks.  Nothing here computes a query result; the oracle binding and the
CUDA binding each translate these descriptions into their own structures.

Readings fixed here (the benchmark description leaves them open):
  * U[a,b] includes both ends.
  * The date dimension is the first 2,556 calendar days from 1992-01-01;
    year = key // 10000; a fact date is the key of a uniformly drawn row.
  * Dimension row r (0-based) of a dense-key dimension has key r + 1.
  * Config 1 filters the date dimension to the year 1993.
  * Config 4: fact columns p U[0,9999], fk, g U[0,2^30-1], m U[0,10^6];
    predicate p < T; the unfiltered 3M-row dimension carries w U[0,3];
    aggregate = sum(m + w) and count per group g % G.
  * Config 5: dimension key = mix(key_seed + r), attr U[0,63],
    payload U[0,2^20-1]; fact fk follows Zipf(1.0) by integer weights.
"""
from __future__ import annotations

from dataclasses import dataclass, field, replace
from typing import Optional

import numpy as np

from . import (DATE_FK_I32, DATE_KEY_I32, DATE_ROWS, DATE_YEAR_I32, MIXKEY_I64, SEQ_I32, UNIFORM_DIV_I32,
               UNIFORM_I32, ZIPF_FK_I64, fill_device, fill_host)

MASTER_SEED = 20260707
C5_KEY_SEED = 0x5EEDC0DE12345678


@dataclass(frozen=True)
class ColSpec:
    name: str
    kind: int
    column_id: int = 0
    a: int = 0
    b: int = 0
    div: int = 1
    key_seed: int = 0
    zipf_k: int = 0

    @property
    def is64(self) -> bool:
        return self.kind in (MIXKEY_I64, ZIPF_FK_I64)


@dataclass(frozen=True)
class Pred:
    col: str
    op: str  # EQ NE LT LE GT GE BETWEEN IN
    lo: int = 0
    hi: int = 0
    values: tuple = ()


@dataclass(frozen=True)
class Term:
    src: str  # "FACT" (a = fact column name) or "PAYLOAD" (a = join index, b = payload index)
    a: object
    b: int = 0
    mult: int = 1


@dataclass(frozen=True)
class KeyExpr:
    terms: tuple
    offset: int = 0
    modulo: int = 0  # 0 = none


@dataclass(frozen=True)
class AggExpr:
    op: str  # COL MUL SUB ADD
    x: Term
    y: Optional[Term] = None
    want_count: bool = True


@dataclass(frozen=True)
class DimSpec:
    name: str
    rows: int
    cols: tuple
    key: str
    preds: tuple = ()
    payloads: tuple = ()
    force_hash: bool = False


@dataclass(frozen=True)
class Workload:
    name: str
    n_rows: int
    fact_cols: tuple
    dims: tuple
    joins: tuple  # (fk fact column name, dim name)
    preds: tuple
    key: Optional[KeyExpr]
    agg: AggExpr
    mode: str  # SCALAR DENSE HASHED
    num_groups: int = 1
    capacity: int = 0
    seed: int = MASTER_SEED
    notes: str = ""

    def fact_col(self, name: str) -> ColSpec:
        for c in self.fact_cols:
            if c.name == name:
                return c
        raise KeyError(name)

    def dim(self, name: str) -> DimSpec:
        for d in self.dims:
            if d.name == name:
                return d
        raise KeyError(name)

    def referenced_bytes_per_row(self) -> int:
        return sum(8 if c.is64 else 4 for c in self.fact_cols)


# ----------------------------------------------------------------------------
# materialisation
# ----------------------------------------------------------------------------
def host_column(seed: int, c: ColSpec, row0: int, n: int) -> np.ndarray:
    return fill_host(c.kind, seed, c.column_id, row0, n, c.a, c.b, c.div, c.key_seed, c.zipf_k)


def device_column(seed: int, c: ColSpec, row0: int, n: int, device="cuda:0"):
    return fill_device(c.kind, seed, c.column_id, row0, n, c.a, c.b, c.div, c.key_seed, c.zipf_k, device=device)


def host_fact(w: Workload, row0: int = 0, n: Optional[int] = None) -> dict:
    n = w.n_rows - row0 if n is None else n
    return {c.name: host_column(w.seed, c, row0, n) for c in w.fact_cols}


def device_fact(w: Workload, row0: int = 0, n: Optional[int] = None, device="cuda:0") -> dict:
    n = w.n_rows - row0 if n is None else n
    return {c.name: device_column(w.seed, c, row0, n, device) for c in w.fact_cols}


def host_dim(w: Workload, d: DimSpec) -> dict:
    return {c.name: host_column(w.seed, c, 0, d.rows) for c in d.cols}


def device_dim(w: Workload, d: DimSpec, device="cuda:0") -> dict:
    return {c.name: device_column(w.seed, c, 0, d.rows, device) for c in d.cols}


# ----------------------------------------------------------------------------
# the five benchmark configurations
# ----------------------------------------------------------------------------
def _date_dim(preds=(), payloads=()) -> DimSpec:
    return DimSpec("date", DATE_ROWS,
                   (ColSpec("datekey", DATE_KEY_I32), ColSpec("year", DATE_YEAR_I32)),
                   key="datekey", preds=tuple(preds), payloads=tuple(payloads))


def config1(n: int = 6_000_000) -> Workload:
    """Filter + scalar aggregate over four fact columns with a date-table probe."""
    base = 100
    fact = (ColSpec("orderdate", DATE_FK_I32, base + 0),
            ColSpec("discount", UNIFORM_I32, base + 1, 0, 10),
            ColSpec("quantity", UNIFORM_I32, base + 2, 1, 50),
            ColSpec("extendedprice", UNIFORM_I32, base + 3, 90000, 10000000))
    date = _date_dim(preds=(Pred("year", "EQ", 1993),))
    return Workload("c1_filter_agg", n, fact, (date,), (("orderdate", "date"),),
                    (Pred("discount", "BETWEEN", 2, 4), Pred("quantity", "LT", 30)),
                    None, AggExpr("MUL", Term("FACT", "extendedprice"), Term("FACT", "discount")), "SCALAR")


def config2(n: int = 60_000_000) -> Workload:
    """Two filtering joins + a date join, group by (year, brand), dense result."""
    base = 200
    fact = (ColSpec("partkey", UNIFORM_I32, base + 0, 1, 200000),
            ColSpec("suppkey", UNIFORM_I32, base + 1, 1, 20000),
            ColSpec("orderdate", DATE_FK_I32, base + 2),
            ColSpec("revenue", UNIFORM_I32, base + 3, 100000, 10000000))
    part = DimSpec("part", 200000,
                   (ColSpec("partkey", SEQ_I32), ColSpec("category", UNIFORM_I32, base + 50, 0, 24),
                    ColSpec("brand", UNIFORM_I32, base + 51, 0, 999)),
                   key="partkey", preds=(Pred("category", "EQ", 7),), payloads=("brand",))
    supp = DimSpec("supplier", 20000,
                   (ColSpec("suppkey", SEQ_I32), ColSpec("region", UNIFORM_I32, base + 60, 0, 4)),
                   key="suppkey", preds=(Pred("region", "EQ", 2),))
    date = _date_dim(payloads=("year",))
    key = KeyExpr((Term("PAYLOAD", 2, 0, 1000), Term("PAYLOAD", 0, 0, 1)), offset=-1992 * 1000)
    return Workload("c2_two_join_groupby", n, fact, (part, supp, date),
                    (("partkey", "part"), ("suppkey", "supplier"), ("orderdate", "date")), (),
                    key, AggExpr("COL", Term("FACT", "revenue")), "DENSE", num_groups=7000)


def config3(n: int = 600_000_000) -> Workload:
    """Four joins, group by (year, customer nation), sum(revenue - supplycost)."""
    base = 300
    fact = (ColSpec("custkey", UNIFORM_I32, base + 0, 1, 3000000),
            ColSpec("suppkey", UNIFORM_I32, base + 1, 1, 200000),
            ColSpec("partkey", UNIFORM_I32, base + 2, 1, 1400000),
            ColSpec("orderdate", DATE_FK_I32, base + 3),
            ColSpec("revenue", UNIFORM_I32, base + 4, 100000, 10000000),
            ColSpec("supplycost", UNIFORM_I32, base + 5, 100000, 10000000))
    cust = DimSpec("customer", 3000000,
                   (ColSpec("custkey", SEQ_I32), ColSpec("nation", UNIFORM_I32, base + 50, 0, 24),
                    ColSpec("region", UNIFORM_DIV_I32, base + 50, 0, 24, div=5)),
                   key="custkey", preds=(Pred("region", "EQ", 1),), payloads=("nation",))
    supp = DimSpec("supplier", 200000,
                   (ColSpec("suppkey", SEQ_I32), ColSpec("nation", UNIFORM_I32, base + 60, 0, 24),
                    ColSpec("region", UNIFORM_DIV_I32, base + 60, 0, 24, div=5)),
                   key="suppkey", preds=(Pred("region", "EQ", 1),))
    part = DimSpec("part", 1400000,
                   (ColSpec("partkey", SEQ_I32), ColSpec("mfgr", UNIFORM_I32, base + 70, 0, 4)),
                   key="partkey", preds=(Pred("mfgr", "IN", values=(0, 1)),))
    date = _date_dim(preds=(Pred("year", "BETWEEN", 1997, 1998),), payloads=("year",))
    key = KeyExpr((Term("PAYLOAD", 3, 0, 25), Term("PAYLOAD", 0, 0, 1)), offset=-1992 * 25)
    return Workload("c3_four_join_groupby", n, fact, (cust, supp, part, date),
                    (("custkey", "customer"), ("suppkey", "supplier"), ("partkey", "part"), ("orderdate", "date")),
                    (), key, AggExpr("SUB", Term("FACT", "revenue"), Term("FACT", "supplycost")), "DENSE",
                    num_groups=175)


C4_THRESHOLDS = {0.0001: 1, 0.01: 100, 0.1: 1000, 0.5: 5000, 1.0: 10000}
C4_GROUPS = (1, 1000, 100000, 1000000)


def config4(n: int = 600_000_000, selectivity: float = 0.1, groups: int = 1000,
            hashed: Optional[bool] = None, dim_rows: int = 3_000_000) -> Workload:
    """One join into an unfiltered dimension; fact predicate p < T; group by g % G."""
    base = 400
    T = C4_THRESHOLDS[selectivity]
    if hashed is None:
        hashed = groups >= 100000
    fact = (ColSpec("p", UNIFORM_I32, base + 0, 0, 9999),
            ColSpec("fk", UNIFORM_I32, base + 1, 1, dim_rows),
            ColSpec("g", UNIFORM_I32, base + 2, 0, (1 << 30) - 1),
            ColSpec("m", UNIFORM_I32, base + 3, 0, 1000000))
    dim = DimSpec("dim", dim_rows, (ColSpec("key", SEQ_I32), ColSpec("w", UNIFORM_I32, base + 50, 0, 3)),
                  key="key", payloads=("w",))
    key = KeyExpr((Term("FACT", "g"),), modulo=groups)
    return Workload(f"c4_sweep_s{selectivity:g}_g{groups}{'_hashed' if hashed else '_dense'}", n, fact, (dim,),
                    (("fk", "dim"),), (Pred("p", "LT", T),), key,
                    AggExpr("ADD", Term("FACT", "m"), Term("PAYLOAD", 0, 0)),
                    "HASHED" if hashed else "DENSE", num_groups=groups, capacity=2 * groups)


def config5(n: int = 300_000_000, dim_rows: int = 8_000_000) -> Workload:
    """Zipf-skewed int64 foreign key into sparse random 64-bit keys; hash probe."""
    base = 500
    fact = (ColSpec("fk", ZIPF_FK_I64, base + 0, key_seed=C5_KEY_SEED, zipf_k=dim_rows),
            ColSpec("measure", UNIFORM_I32, base + 1, 0, 1000000))
    dim = DimSpec("dim", dim_rows,
                  (ColSpec("key", MIXKEY_I64, key_seed=C5_KEY_SEED), ColSpec("attr", UNIFORM_I32, base + 50, 0, 63),
                   ColSpec("payload", UNIFORM_I32, base + 51, 0, (1 << 20) - 1)),
                  key="key", preds=(Pred("attr", "LT", 16),), payloads=("payload",), force_hash=True)
    key = KeyExpr((Term("PAYLOAD", 0, 0),), modulo=4096)
    return Workload("c5_skewed_sparse", n, fact, (dim,), (("fk", "dim"),), (), key,
                    AggExpr("COL", Term("FACT", "measure")), "DENSE", num_groups=4096)


def city_pair(n: int = 600_000_000) -> Workload:
    """Beyond the five benchmark configurations: the paper's city x city shape (Section 3.3: hundreds of
    thousands of groups, few survivors, global group table).  Customer and supplier each carry a city
    U[0,249] and a nation = city // 10; both are filtered to one nation; group by (customer city,
    supplier city, year) = 250 * 250 * 7 = 437,500 dense groups; sum(revenue)."""
    base = 600
    fact = (ColSpec("custkey", UNIFORM_I32, base + 0, 1, 3000000),
            ColSpec("suppkey", UNIFORM_I32, base + 1, 1, 200000),
            ColSpec("orderdate", DATE_FK_I32, base + 2),
            ColSpec("revenue", UNIFORM_I32, base + 3, 100000, 10000000))
    cust = DimSpec("customer", 3000000,
                   (ColSpec("custkey", SEQ_I32), ColSpec("city", UNIFORM_I32, base + 50, 0, 249),
                    ColSpec("nation", UNIFORM_DIV_I32, base + 50, 0, 249, div=10)),
                   key="custkey", preds=(Pred("nation", "EQ", 7),), payloads=("city",))
    supp = DimSpec("supplier", 200000,
                   (ColSpec("suppkey", SEQ_I32), ColSpec("city", UNIFORM_I32, base + 60, 0, 249),
                    ColSpec("nation", UNIFORM_DIV_I32, base + 60, 0, 249, div=10)),
                   key="suppkey", preds=(Pred("nation", "EQ", 7),), payloads=("city",))
    date = _date_dim(payloads=("year",))
    key = KeyExpr((Term("PAYLOAD", 0, 0, 250 * 7), Term("PAYLOAD", 1, 0, 7), Term("PAYLOAD", 2, 0, 1)), offset=-1992)
    return Workload("city_pair_groupby", n, fact, (cust, supp, date),
                    (("custkey", "customer"), ("suppkey", "supplier"), ("orderdate", "date")), (), key,
                    AggExpr("COL", Term("FACT", "revenue")), "DENSE", num_groups=250 * 250 * 7)


def city_brand(n: int = 600_000_000, hashed: bool = True) -> Workload:
    """Beyond the five benchmark configurations: the paper's city x brand shape (Section 3.3, the Q4.3
    pattern: group by year, supplier city and part brand; very few rows survive).  Customer is filtered
    to one region and gathers nothing; supplier is filtered to one nation and gathers its city U[0,249];
    part is filtered to one category and gathers its brand U[0,999]; the date table keeps 1997-1998 and
    gathers the year.  Key ((year - 1992) * 250 + city) * 1000 + brand: 1,750,000 possible groups, of which
    at most 2 * 10 * 1000 can occur; about n / 10,900 rows survive.  sum(revenue - supplycost) and count.
    Asked for as a hashed list (capacity 32,768) by default, or as the dense array of all possible groups."""
    base = 700
    fact = (ColSpec("custkey", UNIFORM_I32, base + 0, 1, 3000000),
            ColSpec("suppkey", UNIFORM_I32, base + 1, 1, 200000),
            ColSpec("partkey", UNIFORM_I32, base + 2, 1, 1400000),
            ColSpec("orderdate", DATE_FK_I32, base + 3),
            ColSpec("revenue", UNIFORM_I32, base + 4, 100000, 10000000),
            ColSpec("supplycost", UNIFORM_I32, base + 5, 100000, 10000000))
    cust = DimSpec("customer", 3000000,
                   (ColSpec("custkey", SEQ_I32), ColSpec("nation", UNIFORM_I32, base + 50, 0, 24),
                    ColSpec("region", UNIFORM_DIV_I32, base + 50, 0, 24, div=5)),
                   key="custkey", preds=(Pred("region", "EQ", 1),))
    supp = DimSpec("supplier", 200000,
                   (ColSpec("suppkey", SEQ_I32), ColSpec("city", UNIFORM_I32, base + 60, 0, 249),
                    ColSpec("nation", UNIFORM_DIV_I32, base + 60, 0, 249, div=10)),
                   key="suppkey", preds=(Pred("nation", "EQ", 7),), payloads=("city",))
    part = DimSpec("part", 1400000,
                   (ColSpec("partkey", SEQ_I32), ColSpec("category", UNIFORM_I32, base + 70, 0, 24),
                    ColSpec("brand", UNIFORM_I32, base + 71, 0, 999)),
                   key="partkey", preds=(Pred("category", "EQ", 3),), payloads=("brand",))
    date = _date_dim(preds=(Pred("year", "BETWEEN", 1997, 1998),), payloads=("year",))
    key = KeyExpr((Term("PAYLOAD", 3, 0, 250 * 1000), Term("PAYLOAD", 1, 0, 1000), Term("PAYLOAD", 2, 0, 1)),
                  offset=-1992 * 250 * 1000)
    return Workload("city_brand_groupby" + ("" if hashed else "_dense"), n, fact, (cust, supp, part, date),
                    (("custkey", "customer"), ("suppkey", "supplier"), ("partkey", "part"), ("orderdate", "date")),
                    (), key, AggExpr("SUB", Term("FACT", "revenue"), Term("FACT", "supplycost")),
                    "HASHED" if hashed else "DENSE", num_groups=7 * 250 * 1000, capacity=32768)


def with_rows(w: Workload, n: int) -> Workload:
    return replace(w, n_rows=n)


CONFIGS = {"c1": config1, "c2": config2, "c3": config3, "c4": config4, "c5": config5}
# star-join shapes beyond the five configurations (the paper's high-cardinality group-bys, Section 3.3)
EXTRA_SHAPES = {"city_pair": city_pair, "city_brand": city_brand}
