"""ctypes binding of the CPU test oracle (oracle/sjq_oracle.cpp).

TEST INFRASTRUCTURE ONLY: imported by tests, by the smoke check and by the
benchmark's CPU-baseline leg.  It never imports the CUDA package.
"""
from __future__ import annotations

import ctypes
import os
import subprocess

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB = os.path.join(_HERE, "libsjq_oracle.so")

OPS = {"EQ": 0, "NE": 1, "LT": 2, "LE": 3, "GT": 4, "GE": 5, "BETWEEN": 6, "IN": 7}
AGGS = {"COL": 0, "MUL": 1, "SUB": 2, "ADD": 3}
MODES = {"SCALAR": 0, "DENSE": 1, "HASHED": 2}
OK, DUP_KEY, GROUP_RANGE, INVALID = 0, 1, 2, 3


class OracleError(RuntimeError):
    def __init__(self, status):
        super().__init__({1: "duplicate dimension key", 2: "group key outside dense range", 3: "invalid"}.get(
            status, str(status)))
        self.status = status


def build(force: bool = False) -> str:
    src = os.path.join(_HERE, "sjq_oracle.cpp")
    if force or not os.path.exists(LIB) or os.path.getmtime(LIB) < os.path.getmtime(src):
        subprocess.check_call(["g++", "-O2", "-std=c++17", "-fPIC", "-shared", "-Wall", "-o", LIB, src], cwd=_HERE)
    return LIB


class _Col(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("is64", ctypes.c_int32), ("n", ctypes.c_int64)]


class _Pred(ctypes.Structure):
    _fields_ = [("col", ctypes.c_int32), ("op", ctypes.c_int32), ("lo", ctypes.c_int64), ("hi", ctypes.c_int64),
                ("set", ctypes.POINTER(ctypes.c_int64)), ("nset", ctypes.c_int32)]


class _Term(ctypes.Structure):
    _fields_ = [("src", ctypes.c_int32), ("a", ctypes.c_int32), ("b", ctypes.c_int32), ("mult", ctypes.c_int64)]


class _Key(ctypes.Structure):
    _fields_ = [("t", _Term * 4), ("nterms", ctypes.c_int32), ("offset", ctypes.c_int64),
                ("modulo", ctypes.c_int64)]


class _Agg(ctypes.Structure):
    _fields_ = [("op", ctypes.c_int32), ("x", _Term), ("y", _Term), ("want_count", ctypes.c_int32)]


class _Join(ctypes.Structure):
    _fields_ = [("fk_col", ctypes.c_int32), ("dim", ctypes.c_void_p)]


_lib = None


def lib():
    global _lib
    if _lib is None:
        L = ctypes.CDLL(build())
        L.orc_dim_build.restype = ctypes.c_void_p
        L.orc_dim_build.argtypes = [ctypes.POINTER(_Col), ctypes.c_int, ctypes.POINTER(_Pred), ctypes.c_int,
                                    ctypes.c_int, ctypes.POINTER(ctypes.c_int), ctypes.c_int,
                                    ctypes.POINTER(ctypes.c_int)]
        L.orc_dim_size.restype = ctypes.c_int64
        L.orc_dim_size.argtypes = [ctypes.c_void_p]
        L.orc_dim_free.argtypes = [ctypes.c_void_p]
        L.orc_run.restype = ctypes.c_void_p
        L.orc_run.argtypes = [ctypes.POINTER(_Col), ctypes.c_int, ctypes.c_int64, ctypes.c_int64,
                              ctypes.POINTER(_Pred), ctypes.c_int, ctypes.POINTER(_Join), ctypes.c_int,
                              ctypes.POINTER(_Key), ctypes.POINTER(_Agg), ctypes.c_int, ctypes.c_int64,
                              ctypes.POINTER(ctypes.c_int), ctypes.POINTER(ctypes.c_double)]
        L.orc_result_groups.restype = ctypes.c_int64
        L.orc_result_groups.argtypes = [ctypes.c_void_p]
        L.orc_result_copy.argtypes = [ctypes.c_void_p] + [ctypes.c_void_p] * 3
        L.orc_result_free.argtypes = [ctypes.c_void_p]
        _lib = L
    return _lib


def _cols(names, arrays):
    keep = []
    out = (_Col * len(names))()
    for i, nm in enumerate(names):
        a = np.ascontiguousarray(arrays[nm])
        assert a.dtype in (np.int32, np.int64), a.dtype
        keep.append(a)
        out[i] = _Col(a.ctypes.data, 1 if a.dtype == np.int64 else 0, a.size)
    return out, keep


def _preds(preds, names):
    keep = []
    out = (_Pred * max(1, len(preds)))()
    for i, p in enumerate(preds):
        vals = (ctypes.c_int64 * max(1, len(p.values)))(*p.values)
        keep.append(vals)
        out[i] = _Pred(names.index(p.col), OPS[p.op], p.lo, p.hi, vals, len(p.values))
    return out, keep


class Dim:
    """A filtered dimension held by the oracle (key -> payload tuple)."""

    def __init__(self, spec, arrays):
        names = [c.name for c in spec.cols]
        cols, self._keep = _cols(names, arrays)
        preds, keep2 = _preds(spec.preds, names)
        pay = (ctypes.c_int * max(1, len(spec.payloads)))(*[names.index(p) for p in spec.payloads])
        st = ctypes.c_int(0)
        self.ptr = lib().orc_dim_build(cols, len(names), preds, len(spec.preds), names.index(spec.key), pay,
                                       len(spec.payloads), ctypes.byref(st))
        self.status = st.value
        self.entries = lib().orc_dim_size(self.ptr)

    def __del__(self):
        if getattr(self, "ptr", None):
            lib().orc_dim_free(self.ptr)
            self.ptr = None


def _term(t, fact_names):
    if t is None:
        return _Term(0, 0, 0, 0)
    if t.src == "FACT":
        return _Term(0, fact_names.index(t.a), 0, t.mult)
    return _Term(1, int(t.a), t.b, t.mult)


def run(w, fact: dict, dims: dict, row_begin: int = 0, row_end: int | None = None, check: bool = True):
    """Evaluate workload `w` over host columns `fact` with oracle dimensions
    `dims` (name -> Dim).  Returns a dict: mode SCALAR -> sum,count;
    DENSE -> sums[num_groups], counts[num_groups]; HASHED -> keys, sums,
    counts in ascending key order.  Also 'seconds' (row loop only) and 'status'."""
    names = [c.name for c in w.fact_cols]
    cols, keep = _cols(names, fact)
    n = keep[0].size
    row_end = n if row_end is None else row_end
    preds, keep2 = _preds(w.preds, names)
    joins = (_Join * max(1, len(w.joins)))()
    for j, (fk, dname) in enumerate(w.joins):
        if check and dims[dname].status != OK:
            raise OracleError(dims[dname].status)
        joins[j] = _Join(names.index(fk), dims[dname].ptr)
    key = _Key()
    if w.key is not None:
        assert len(w.key.terms) <= 4
        for i, t in enumerate(w.key.terms):
            key.t[i] = _term(t, names)
        key.nterms, key.offset, key.modulo = len(w.key.terms), w.key.offset, w.key.modulo
    agg = _Agg(AGGS[w.agg.op], _term(w.agg.x, names), _term(w.agg.y, names), int(w.agg.want_count))
    st = ctypes.c_int(0)
    secs = ctypes.c_double(0.0)
    r = lib().orc_run(cols, len(names), row_begin, row_end, preds, len(w.preds), joins, len(w.joins),
                      ctypes.byref(key) if w.key is not None else None, ctypes.byref(agg), MODES[w.mode],
                      w.num_groups, ctypes.byref(st), ctypes.byref(secs))
    try:
        if check and st.value != OK:
            raise OracleError(st.value)
        g = lib().orc_result_groups(r)
        keys = np.empty(g, np.int64)
        sums = np.empty(g, np.int64)
        counts = np.empty(g, np.int64)
        lib().orc_result_copy(r, keys.ctypes.data, sums.ctypes.data, counts.ctypes.data)
    finally:
        lib().orc_result_free(r)
    out = {"seconds": secs.value, "status": st.value}
    if w.mode == "SCALAR":
        out["sum"] = int(sums[0]) if g else 0
        out["count"] = int(counts[0]) if g else 0
    elif w.mode == "DENSE":
        ds = np.zeros(w.num_groups, np.int64)
        dc = np.zeros(w.num_groups, np.int64)
        ds[keys] = sums
        dc[keys] = counts
        out["sums"], out["counts"] = ds, dc
    else:
        out["keys"], out["sums"], out["counts"] = keys, sums, counts
    return out


def build_dims(w, host_dims: dict) -> dict:
    """host_dims: dim name -> dict of numpy columns."""
    return {d.name: Dim(d, host_dims[d.name]) for d in w.dims}
