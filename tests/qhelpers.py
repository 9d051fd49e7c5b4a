"""Helpers shared by the CPU and GPU tests: ad-hoc workloads over explicit
arrays and a seeded random small-query generator (inputs only; no query
arithmetic)."""
import json
import os

import numpy as np

from datagen import MIXKEY_I64, UNIFORM_I32
from datagen.workloads import AggExpr, ColSpec, DimSpec, KeyExpr, Pred, Term, Workload

GOLDEN = os.path.join(os.path.dirname(os.path.abspath(__file__)), "golden")


def golden(name):
    with open(os.path.join(GOLDEN, name)) as f:
        return json.load(f)


def colspecs(arrays):
    return tuple(ColSpec(nm, MIXKEY_I64 if np.asarray(a).dtype == np.int64 else UNIFORM_I32)
                 for nm, a in arrays.items())


def arrays32(d, wide=()):
    return {k: np.asarray(v, dtype=np.int64 if k in wide else np.int32) for k, v in d.items()}


def adhoc(name, fact, dims, joins, preds, key, agg, mode, num_groups=1, capacity=0):
    """dims: list of (name, arrays, key, preds, payloads[, force_hash])."""
    dspecs = []
    for d in dims:
        nm, arr, k, dp, pay = d[:5]
        fh = d[5] if len(d) > 5 else False
        dspecs.append(DimSpec(nm, len(arr[k]), colspecs(arr), key=k, preds=tuple(dp), payloads=tuple(pay),
                              force_hash=fh))
    n = len(next(iter(fact.values())))
    return Workload(name, n, colspecs(fact), tuple(dspecs), tuple(joins), tuple(preds), key, agg, mode,
                    num_groups=num_groups, capacity=capacity)


def ex1():
    g = golden("ex1_filter_scalar.json")
    fact = arrays32(g["fact"])
    date = arrays32(g["date"])
    w = adhoc("ex1", fact, [("date", date, "datekey", [Pred("year", "EQ", 1993)], [])], [("orderdate", "date")],
              [Pred("discount", "BETWEEN", 2, 4), Pred("quantity", "LT", 30)], None,
              AggExpr("MUL", Term("FACT", "extendedprice"), Term("FACT", "discount")), "SCALAR")
    return w, fact, {"date": date}, g["expected"]


def ex2():
    g = golden("ex2_two_join_groupby.json")
    fact = arrays32(g["fact"])
    dims = {k: arrays32(g[k]) for k in ("part", "supplier", "date")}
    key = KeyExpr((Term("PAYLOAD", 2, 0, 1000), Term("PAYLOAD", 0, 0, 1)), offset=-1992 * 1000)
    w = adhoc("ex2", fact,
              [("part", dims["part"], "partkey", [Pred("category", "EQ", 7)], ["brand"]),
               ("supplier", dims["supplier"], "suppkey", [Pred("region", "EQ", 2)], []),
               ("date", dims["date"], "datekey", [], ["year"])],
              [("partkey", "part"), ("suppkey", "supplier"), ("orderdate", "date")], [], key,
              AggExpr("COL", Term("FACT", "revenue")), "DENSE", num_groups=7000)
    return w, fact, dims, {int(k): v for k, v in g["expected"].items()}


def ex3():
    g = golden("ex3_int64_hashed.json")
    fact = arrays32(g["fact"], wide=("fk",))
    dim = arrays32(g["dim"], wide=("key",))
    key = KeyExpr((Term("PAYLOAD", 0, 0, 2),), offset=1, modulo=5)
    w = adhoc("ex3", fact, [("dim", dim, "key", [Pred("attr", "LE", 3)], ["pay"], True)], [("fk", "dim")], [], key,
              AggExpr("MUL", Term("FACT", "m"), Term("PAYLOAD", 0, 0, 3)), "HASHED", capacity=16)
    return w, fact, {"dim": dim}, {int(k): v for k, v in g["expected"].items()}


OPS = ("EQ", "NE", "LT", "LE", "GT", "GE", "BETWEEN", "IN")


def _rand_pred(rng, col, lo, hi):
    op = OPS[rng.integers(len(OPS))]
    a, b = sorted(int(x) for x in rng.integers(lo, hi + 1, 2))
    if op == "IN":
        vals = tuple(int(x) for x in rng.integers(lo, hi + 1, rng.integers(1, 5)))
        return Pred(col, "IN", values=vals)
    return Pred(col, op, a, b)


def random_query(seed, n_fact=48, max_dim=12, allow_dup=False, wide_keys=False, n_joins=None, mode=None):
    """A random tiny star-join query with 0-4 joins, random predicates of every
    operator, and a random result mode.  Returns (workload, fact, host_dims)."""
    rng = np.random.default_rng(seed)
    nj = int(rng.integers(0, 5)) if n_joins is None else n_joins
    fact = {}
    dims = []
    joins = []
    host_dims = {}
    for j in range(nj):
        rows = int(rng.integers(1, max_dim + 1))
        wide = wide_keys and rng.integers(2) == 1
        if wide:
            pool = rng.integers(-(1 << 62), 1 << 62, rows + 4)
        else:
            base = int(rng.integers(-5, 50))
            pool = base + rng.permutation(rows + 4)
        keys = pool[:rows].copy()
        if allow_dup and rows > 1 and rng.integers(3) == 0:
            keys[-1] = keys[0]
        npay = int(rng.integers(0, 3))
        arr = {"k": keys.astype(np.int64 if wide else np.int32),
               "f": rng.integers(0, 4, rows).astype(np.int32)}
        for p in range(npay):
            arr[f"p{p}"] = rng.integers(-3 if p else 0, 9, rows).astype(np.int32)
        dp = [_rand_pred(rng, "f", 0, 3)] if rng.integers(3) == 0 else []
        name = f"d{j}"
        dims.append((name, arr, "k", dp, [f"p{p}" for p in range(npay)], bool(wide or rng.integers(4) == 0)))
        host_dims[name] = arr
        pick = np.where(rng.random(n_fact) < 0.85, rng.integers(0, rows, n_fact), rng.integers(0, rows + 4, n_fact))
        fk = pool[pick]
        fact[f"fk{j}"] = fk.astype(np.int64 if wide else np.int32)
        joins.append((f"fk{j}", name))
    for c in range(3):
        fact[f"c{c}"] = rng.integers(-4, 12, n_fact).astype(np.int32)
    fact["v64"] = rng.integers(-(1 << 40), 1 << 40, n_fact).astype(np.int64)
    preds = [_rand_pred(rng, f"c{c}", -4, 11) for c in range(3) if rng.integers(3) == 0]
    # terms available to the key and the aggregate
    avail = [Term("FACT", f"c{c}", 0, int(rng.integers(-3, 4)) or 1) for c in range(3)]
    avail.append(Term("FACT", "v64", 0, 1))
    for j, d in enumerate(dims):
        for p in range(len(d[4])):
            avail.append(Term("PAYLOAD", j, p, int(rng.integers(-2, 5)) or 1))
    mode = mode or ("SCALAR", "DENSE", "HASHED")[rng.integers(3)]
    key = None
    G = 1
    if mode != "SCALAR":
        nt = int(rng.integers(1, 4))
        terms = tuple(avail[i] for i in rng.integers(0, len(avail), nt))
        if mode == "DENSE":
            G = int(rng.integers(1, 40))
            key = KeyExpr(terms, offset=int(rng.integers(0, 100)), modulo=G if rng.integers(4) else 0)
        else:
            key = KeyExpr(terms, offset=int(rng.integers(-50, 50)),
                          modulo=int(rng.integers(1, 30)) if rng.integers(2) else 0)
    op = ("COL", "MUL", "SUB", "ADD")[rng.integers(4)]
    x = avail[rng.integers(len(avail))]
    y = avail[rng.integers(len(avail))] if op != "COL" else None
    agg = AggExpr(op, x, y, True)
    w = adhoc(f"rand{seed}", fact, dims, joins, preds, key, agg, mode, num_groups=G, capacity=4 * n_fact + 16)
    return w, fact, host_dims
