"""ctypes binding of the C ABI declared in include/sjq.h.

Only argument marshalling happens here: every step of the query runs in the
CUDA kernels of libsjq.so.  PyTorch supplies device memory and the stream.
There is no CPU fallback: if the library is missing, importing fails.
"""
from __future__ import annotations

import ctypes
import os
from dataclasses import dataclass, field, replace
from typing import Optional, Sequence

import torch

_HERE = os.path.dirname(os.path.abspath(__file__))
LIB_PATH = os.path.join(_HERE, "libsjq.so")

MAX_PREDS, MAX_JOINS, MAX_PAYLOADS, MAX_KEY_TERMS = 16, 8, 2, 4
PLAN_SCRATCH_BYTES = 256
OPS = {"EQ": 0, "NE": 1, "LT": 2, "LE": 3, "GT": 4, "GE": 5, "BETWEEN": 6, "IN": 7}
AGGS = {"COL": 0, "MUL": 1, "SUB": 2, "ADD": 3}
MODES = {"SCALAR": 0, "DENSE": 1, "HASHED": 2}
TABLE_KINDS = {1: "DIRECT_BITMAP", 2: "DIRECT_U8", 3: "DIRECT_U16", 4: "DIRECT_U32", 5: "DIRECT_U64", 6: "HASH_I32",
               7: "HASH_I64", 8: "DIRECT_U4", 9: "DIRECT_U2"}
HASH_KINDS = (6, 7)
FORCE_DIRECT, FORCE_HASH = 100, 101
AGG_PATHS = {0: "registers", 1: "shared", 2: "global", 3: "hash"}


class SjqError(RuntimeError):
    def __init__(self, status: int, where: str = ""):
        self.status = int(status)
        super().__init__(f"{where}: {strerror(status)} ({status})")


class _Col(ctypes.Structure):
    _fields_ = [("data", ctypes.c_void_p), ("dtype", ctypes.c_int32), ("n", ctypes.c_int64)]


class _Pred(ctypes.Structure):
    _fields_ = [("col", ctypes.c_int32), ("op", ctypes.c_int32), ("lo", ctypes.c_int64), ("hi", ctypes.c_int64),
                ("set", ctypes.POINTER(ctypes.c_int64)), ("nset", ctypes.c_int32)]


class _Term(ctypes.Structure):
    _fields_ = [("src", ctypes.c_int32), ("a", ctypes.c_int32), ("b", ctypes.c_int32), ("mult", ctypes.c_int64)]


class _KeyExpr(ctypes.Structure):
    _fields_ = [("t", _Term * MAX_KEY_TERMS), ("nterms", ctypes.c_int32), ("offset", ctypes.c_int64),
                ("modulo", ctypes.c_int64)]


class _AggExpr(ctypes.Structure):
    _fields_ = [("op", ctypes.c_int32), ("x", _Term), ("y", _Term), ("want_count", ctypes.c_int32)]


class _BuildOpts(ctypes.Structure):
    _fields_ = [("force_kind", ctypes.c_int32), ("hash_load_pct", ctypes.c_int32),
                ("max_direct_bytes", ctypes.c_int64), ("min_code_bits", ctypes.c_int32), ("reserved", ctypes.c_int32)]


class DimLayout(ctypes.Structure):
    _fields_ = [("kind", ctypes.c_int32), ("key_dtype", ctypes.c_int32), ("npayload", ctypes.c_int32),
                ("code_bits", ctypes.c_int32), ("dim_rows", ctypes.c_int64), ("entries", ctypes.c_int64),
                ("kmin", ctypes.c_int64), ("kmax", ctypes.c_int64), ("pay_min", ctypes.c_int64 * MAX_PAYLOADS),
                ("pay_max", ctypes.c_int64 * MAX_PAYLOADS), ("pay_bits", ctypes.c_int32 * MAX_PAYLOADS),
                ("slots", ctypes.c_int64), ("filter_bits", ctypes.c_int64), ("table_bytes", ctypes.c_size_t)]

    @property
    def kind_name(self) -> str:
        return TABLE_KINDS.get(self.kind, str(self.kind))


class _Join(ctypes.Structure):
    _fields_ = [("fk_col", ctypes.c_int32), ("table", ctypes.c_void_p)]


class _ResultSpec(ctypes.Structure):
    _fields_ = [("mode", ctypes.c_int32), ("num_groups", ctypes.c_int64), ("capacity", ctypes.c_int64)]


class _Result(ctypes.Structure):
    _fields_ = [("sums", ctypes.c_void_p), ("counts", ctypes.c_void_p), ("keys", ctypes.c_void_p),
                ("n_groups", ctypes.c_void_p), ("status", ctypes.c_void_p), ("workspace", ctypes.c_void_p),
                ("workspace_bytes", ctypes.c_size_t)]


class _RunOpts(ctypes.Structure):
    _fields_ = [("block_threads", ctypes.c_int32), ("ctas_per_sm", ctypes.c_int32), ("eager_loads", ctypes.c_int32),
                ("agg_path", ctypes.c_int32), ("smem_tables", ctypes.c_int32), ("compaction", ctypes.c_int32),
                ("accumulate", ctypes.c_int32), ("norder", ctypes.c_int32),
                ("order", ctypes.c_int32 * (MAX_PREDS + MAX_JOINS)), ("event_before", ctypes.c_void_p),
                ("event_after", ctypes.c_void_p), ("specialise", ctypes.c_int32),
                ("rows_per_lane", ctypes.c_int32), ("no_filter_bitmap", ctypes.c_int32),
                ("host_copy_all", ctypes.c_int32), ("dense_slots", ctypes.c_int32),
                ("group_hash_always", ctypes.c_int32), ("warp_agg", ctypes.c_int32), ("unfused", ctypes.c_int32),
                ("unfused_scratch", ctypes.c_void_p), ("unfused_scratch_bytes", ctypes.c_size_t),
                ("pass_ppm", ctypes.c_int32 * (MAX_PREDS + MAX_JOINS)), ("hot_keys", ctypes.c_int32),
                ("hot_scratch", ctypes.c_void_p), ("hot_scratch_bytes", ctypes.c_size_t), ("l0_bulk", ctypes.c_int32)]


class RunInfo(ctypes.Structure):
    _fields_ = [("nstages", ctypes.c_int32), ("order", ctypes.c_int32 * (MAX_PREDS + MAX_JOINS + 8)),
                ("stage_in_smem", ctypes.c_int32 * (MAX_PREDS + MAX_JOINS + 8)),
                ("first_sparse_stage", ctypes.c_int32), ("reserved_levels", ctypes.c_int32),
                ("agg_path", ctypes.c_int32), ("grid", ctypes.c_int32),
                ("block", ctypes.c_int32), ("smem_bytes", ctypes.c_int32), ("kernel_launches", ctypes.c_int32)]

    def describe(self) -> dict:
        return {"order": list(self.order[: self.nstages]), "in_smem": list(self.stage_in_smem[: self.nstages]),
                "first_sparse_stage": self.first_sparse_stage, "queue_levels": self.reserved_levels, "agg_path": AGG_PATHS.get(self.agg_path),
                "grid": self.grid, "block": self.block, "smem_bytes": self.smem_bytes,
                "kernel_launches": self.kernel_launches}


@dataclass
class RunOpts:
    block_threads: int = 0
    ctas_per_sm: int = 0
    eager_loads: bool = False
    agg_path: int = 0
    smem_tables: int = 0
    compaction: int = 0
    accumulate: bool = False
    order: Sequence[int] = ()
    events: Optional[tuple] = None  # (torch.cuda.Event, torch.cuda.Event), both already recorded once
    specialise: bool = False  # compile the fused kernel for this query's shape at run time (cached per shape)
    rows_per_lane: int = 0  # queue-fed levels: 0 auto, 4, or 8 (8 needs specialise)
    no_filter_bitmap: bool = False  # filter stages probe the code array of a direct table, not its bitmap
    host_copy_all: bool = False  # run_host: copy every referenced column instead of reading sparse ones in place
    dense_slots: int = 0  # level 0: 0 auto, 2, or 4 groups of four rows per thread (4 needs specialise)
    group_hash_always: bool = False  # HASHED: keep the group hash table even when the key domain is small
    warp_agg: int = 0  # group-by terminal: 1 = add equal keys inside the warp before the atomics; 0 / 2 = off
    unfused_scratch: Optional[torch.Tensor] = None  # ablation: run operator at a time with this CUDA uint8 scratch
    pass_ppm: Sequence[int] = ()  # measured pass fractions (parts per million): predicates, then joins; 0 = unknown
    hot_keys: int = 0  # open-addressing joins: 0 auto, 1 hot-key table whenever possible, 2 never
    hot_scratch: Optional[torch.Tensor] = None  # CUDA uint8 scratch of HOT_SCRATCH_BYTES; run() supplies one if None
    l0_bulk: int = 0  # 1 = first column by bulk-asynchronous copies into shared memory when it fits; 0 / 2 = loads

    def to_c(self) -> _RunOpts:
        o = _RunOpts()
        o.block_threads, o.ctas_per_sm = self.block_threads, self.ctas_per_sm
        o.eager_loads, o.agg_path, o.smem_tables = int(self.eager_loads), self.agg_path, self.smem_tables
        o.compaction, o.accumulate = self.compaction, int(self.accumulate)
        o.norder = len(self.order)
        for i, v in enumerate(self.order):
            o.order[i] = v
        for i, v in enumerate(self.pass_ppm):
            o.pass_ppm[i] = int(v)
        o.warp_agg = self.warp_agg
        o.hot_keys = self.hot_keys
        o.l0_bulk = self.l0_bulk
        if self.hot_scratch is not None:
            o.hot_scratch = self.hot_scratch.data_ptr()
            o.hot_scratch_bytes = self.hot_scratch.numel()
        if self.unfused_scratch is not None:
            o.unfused = 1
            o.unfused_scratch = self.unfused_scratch.data_ptr()
            o.unfused_scratch_bytes = self.unfused_scratch.numel()
        o.specialise = int(self.specialise)
        o.rows_per_lane = self.rows_per_lane
        o.no_filter_bitmap = int(self.no_filter_bitmap)
        o.host_copy_all = int(self.host_copy_all)
        o.dense_slots = self.dense_slots
        o.group_hash_always = int(self.group_hash_always)
        if self.events is not None:
            o.event_before, o.event_after = self.events[0].cuda_event, self.events[1].cuda_event
        return o


_lib = None


def lib():
    """Load libsjq.so; raises if it has not been built (no fallback exists)."""
    global _lib
    if _lib is None:
        if not os.path.exists(LIB_PATH):
            raise ImportError(f"{LIB_PATH} is missing: build it with paper_2607_07632_b200/build.py "
                              "(there is no CPU fallback)")
        L = ctypes.CDLL(LIB_PATH)
        vp, ip = ctypes.c_void_p, ctypes.c_int
        L.sjq_dim_plan.restype = ctypes.c_int32
        L.sjq_dim_plan.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip, ip, ctypes.POINTER(ip), ip,
                                   ctypes.POINTER(_BuildOpts), vp, vp, ctypes.POINTER(DimLayout)]
        L.sjq_dim_plan_begin.restype = ctypes.c_int32
        L.sjq_dim_plan_begin.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip, ip, ctypes.POINTER(ip),
                                         ip, vp, vp, vp]
        L.sjq_dim_plan_end.restype = ctypes.c_int32
        L.sjq_dim_plan_end.argtypes = [ctypes.POINTER(_Col), ip, ip, ip, ctypes.POINTER(_BuildOpts), vp,
                                       ctypes.POINTER(DimLayout)]
        L.sjq_build_dim.restype = ctypes.c_int32
        L.sjq_build_dim.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip, ip, ctypes.POINTER(ip), ip,
                                    ctypes.POINTER(DimLayout), vp, ctypes.c_size_t, vp, vp, ctypes.POINTER(vp)]
        L.sjq_dim_layout_bytes.restype = ctypes.c_int32
        L.sjq_dim_layout_bytes.argtypes = [ctypes.POINTER(DimLayout), ctypes.POINTER(ctypes.c_size_t)]
        L.sjq_table_info.restype = ctypes.c_int32
        L.sjq_table_info.argtypes = [vp, ctypes.POINTER(DimLayout)]
        L.sjq_table_destroy.restype = None
        L.sjq_table_destroy.argtypes = [vp]
        L.sjq_pred_sample.restype = ctypes.c_int32
        L.sjq_pred_sample.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip, vp, vp,
                                      ctypes.POINTER(ctypes.c_int32)]
        L.sjq_pred_sample_begin.restype = ctypes.c_int32
        L.sjq_pred_sample_begin.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip, vp, vp, vp]
        L.sjq_pred_sample_end.restype = ctypes.c_int32
        L.sjq_pred_sample_end.argtypes = [vp, ip, ctypes.POINTER(ctypes.c_int32)]
        L.sjq_run_workspace_bytes.restype = ctypes.c_int32
        L.sjq_run_workspace_bytes.argtypes = [ctypes.POINTER(_ResultSpec), ctypes.POINTER(ctypes.c_size_t)]
        L.sjq_run.restype = ctypes.c_int32
        L.sjq_run.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip, ctypes.POINTER(_Join), ip,
                              ctypes.POINTER(_KeyExpr), ctypes.POINTER(_AggExpr), ctypes.POINTER(_ResultSpec),
                              ctypes.POINTER(_Result), ctypes.POINTER(_RunOpts), vp, ctypes.POINTER(RunInfo)]
        L.sjq_run_host.restype = ctypes.c_int32
        L.sjq_run_host.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip, ctypes.POINTER(_Join), ip,
                                   ctypes.POINTER(_KeyExpr), ctypes.POINTER(_AggExpr), ctypes.POINTER(_ResultSpec),
                                   ctypes.POINTER(_Result), ctypes.POINTER(_RunOpts), vp, ctypes.c_size_t,
                                   ctypes.c_int64, vp, vp, vp, vp, vp, vp]
        L.sjq_merge_groups.restype = ctypes.c_int32
        L.sjq_merge_groups.argtypes = [vp, vp, vp, ctypes.c_int64, ctypes.c_int64, ctypes.POINTER(_Result), vp]
        L.sjq_run_hashed_static.restype = ctypes.c_int32
        L.sjq_run_hashed_static.argtypes = [ctypes.POINTER(_Col), ip, ctypes.POINTER(_Pred), ip,
                                            ctypes.POINTER(_Join), ip, ctypes.POINTER(_KeyExpr),
                                            ctypes.POINTER(_AggExpr), ctypes.c_int64, ctypes.POINTER(_Result),
                                            ctypes.POINTER(_RunOpts), vp, ctypes.POINTER(RunInfo)]
        L.sjq_strerror.restype = ctypes.c_char_p
        L.sjq_strerror.argtypes = [ctypes.c_int32]
        L.sjq_version.restype = ctypes.c_char_p
        _lib = L
    return _lib


def strerror(status: int) -> str:
    return lib().sjq_strerror(int(status)).decode()


def version() -> str:
    return lib().sjq_version().decode()


def _stream_ptr(device) -> int:
    return torch.cuda.current_stream(device).cuda_stream


def _cols(tensors: Sequence[torch.Tensor]):
    arr = (_Col * max(1, len(tensors)))()
    for i, t in enumerate(tensors):
        if t.dtype not in (torch.int32, torch.int64) or not t.is_cuda or not t.is_contiguous() or t.dim() != 1:
            raise ValueError("columns must be contiguous 1-D int32/int64 CUDA tensors")
        arr[i] = _Col(t.data_ptr(), 1 if t.dtype == torch.int64 else 0, t.numel())
    return arr


def _preds(preds, names: Sequence[str]):
    keep = []
    arr = (_Pred * max(1, len(preds)))()
    for i, p in enumerate(preds):
        vals = (ctypes.c_int64 * max(1, len(p.values)))(*p.values)
        keep.append(vals)
        arr[i] = _Pred(names.index(p.col), OPS[p.op], p.lo, p.hi, vals, len(p.values))
    return arr, keep


def layout_bytes(layout: DimLayout) -> int:
    """sjq_dim_layout_bytes: device bytes a table of this shape needs (raises if the shape is inconsistent)."""
    n = ctypes.c_size_t(0)
    rc = lib().sjq_dim_layout_bytes(ctypes.byref(layout), ctypes.byref(n))
    if rc != 0:
        raise SjqError(rc, "sjq_dim_layout_bytes")
    return int(n.value)


class Table:
    """A built dimension table: host handle + the device memory it lives in."""

    def __init__(self, handle: int, layout: DimLayout, mem: torch.Tensor, status: torch.Tensor):
        self.handle, self.layout, self.mem, self.status_dev = handle, layout, mem, status

    def status(self) -> int:
        return int(self.status_dev.item())

    def check(self) -> "Table":
        st = self.status()
        if st != 0:
            raise SjqError(st, "sjq_build_dim")
        return self

    def __del__(self):
        if getattr(self, "handle", None) and _lib is not None:
            _lib.sjq_table_destroy(self.handle)
            self.handle = None


def build_dim(cols: dict, key: str, preds=(), payloads=(), force_kind: int = 0, hash_load_pct: int = 0,
              max_direct_bytes: int = 0, edit_layout=None, min_code_bits: int = 0, mem_offset: int = 0) -> Table:
    """sjq_dim_plan + sjq_build_dim over a dict of CUDA tensors (dimension columns).  `edit_layout`, if
    given, is called with the planned DimLayout and may change it before the build (sjq_build_dim takes
    the layout from its caller: tests use this to hand it an undersized or inconsistent one).  `mem_offset`
    (a multiple of 16) places the table that many bytes into its allocation: table memory only has to be
    16-byte aligned, and tests use this to get exactly that."""
    names = list(cols.keys())
    tensors = [cols[n] for n in names]
    device = tensors[0].device
    with torch.cuda.device(device):
        carr = _cols(tensors)
        parr, keep = _preds(preds, names)
        pay = (ctypes.c_int * max(1, len(payloads)))(*[names.index(p) for p in payloads])
        opts = _BuildOpts(force_kind, hash_load_pct, max_direct_bytes, min_code_bits, 0)
        scratch = torch.empty(PLAN_SCRATCH_BYTES, dtype=torch.uint8, device=device)
        layout = DimLayout()
        stream = _stream_ptr(device)
        rc = lib().sjq_dim_plan(carr, len(names), parr, len(preds), names.index(key), pay, len(payloads),
                                ctypes.byref(opts), scratch.data_ptr(), stream, ctypes.byref(layout))
        if rc != 0:
            raise SjqError(rc, "sjq_dim_plan")
        planned_bytes = layout.table_bytes
        if edit_layout is not None:
            edit_layout(layout)
        mem = torch.empty(max(planned_bytes, layout.table_bytes) + mem_offset, dtype=torch.uint8, device=device)[mem_offset:]
        status = torch.zeros(1, dtype=torch.int32, device=device)
        handle = ctypes.c_void_p()
        rc = lib().sjq_build_dim(carr, len(names), parr, len(preds), names.index(key), pay, len(payloads),
                                 ctypes.byref(layout), mem.data_ptr(), mem.numel(), status.data_ptr(), stream,
                                 ctypes.byref(handle))
        if rc != 0:
            raise SjqError(rc, "sjq_build_dim")
    return Table(handle.value, layout, mem, status)


class TableBuilder:
    """A dimension prepared for repeated builds: the argument structures are marshalled once, scratch,
    statistics and table memory are kept, and plan + build run on a side stream so that several
    dimensions can be planned with a single wait (sjq_dim_plan_begin / _end, sjq_build_dim)."""

    def __init__(self, cols: dict, key: str, preds=(), payloads=(), force_kind: int = 0, hash_load_pct: int = 0,
                 max_direct_bytes: int = 0, min_code_bits: int = 0, reuse_layout: bool = False):
        self.names = list(cols.keys())
        self.tensors = [cols[n] for n in self.names]
        self.device = self.tensors[0].device
        # reuse_layout: a repeated build does not wait for its own key-range scan.  It is enqueued with the
        # layout chosen from the newest scan whose statistics have already reached the host (the previous
        # step's, as a rule) and the build kernel checks every key and payload against that layout on the
        # device (SJQ_ERR_LAYOUT_MISMATCH / TABLE_FULL in the table's status word if the dimension outgrew it).
        # A changed dimension is therefore re-planned one or two steps late, never silently mis-built.
        self.reuse_layout = reuse_layout
        self.planned = False
        with torch.cuda.device(self.device):
            self.carr = _cols(self.tensors)
            self.parr, self._keep = _preds(preds, self.names)
            self.npreds, self.npay = len(preds), len(payloads)
            self.key_col = self.names.index(key)
            self.pay = (ctypes.c_int * max(1, len(payloads)))(*[self.names.index(p) for p in payloads])
            self.opts = _BuildOpts(force_kind, hash_load_pct, max_direct_bytes, min_code_bits, 0)
            self.scratch = torch.empty(PLAN_SCRATCH_BYTES, dtype=torch.uint8, device=self.device)
            # statistics of the last few scans (page-locked, written by an asynchronous copy), each with the
            # event that says its copy has landed
            self.stats = [torch.zeros(8, dtype=torch.int64, pin_memory=True) for _ in range(4)]
            self.stats_done = [torch.cuda.Event() for _ in self.stats]
            self.stats_used = [False] * len(self.stats)
            self.scan = -1  # ring position of the newest scan
            self.status = torch.zeros(1, dtype=torch.int32, device=self.device)
            self.side = torch.cuda.Stream(self.device)       # builds
            self.scan_side = torch.cuda.Stream(self.device)  # key-range scans: independent of the builds
            # two table buffers used in turn: the build of the next table does not have to wait for the run
            # that still reads the previous one
            self.mems = [None, None]
            self.turn = 0
            self.guards = [torch.cuda.Event(), torch.cuda.Event()]
            self.guard_set = [False, False]
            self.layout = DimLayout()

    def begin(self):
        """Enqueue the key-range scan on the side stream.  It only reads the dimension columns, so it does
        not wait for work queued on the current stream (a previous run may still be reading the old table)."""
        j = (self.scan + 1) % len(self.stats)
        if self.stats_used[j]:
            self.stats_done[j].synchronize()  # the host is a whole ring ahead of the device
        rc = lib().sjq_dim_plan_begin(self.carr, len(self.names), self.parr, self.npreds, self.key_col, self.pay,
                                      self.npay, self.scratch.data_ptr(), self.stats[j].data_ptr(),
                                      self.scan_side.cuda_stream)
        if rc != 0:
            raise SjqError(rc, "sjq_dim_plan_begin")
        self.stats_done[j].record(self.scan_side)
        self.stats_used[j] = True
        self.scan = j

    def after(self, stream):
        """Scans and builds enqueued from now on follow the work already queued on `stream` (e.g. copies that
        refresh the dimension columns)."""
        self.side.wait_stream(stream)
        self.scan_side.wait_stream(stream)

    def _choose_layout(self):
        """The layout for the scan just enqueued, or (reuse_layout) for the newest one that has completed."""
        n = len(self.stats)
        j = self.scan
        if self.reuse_layout and self.planned:
            for back in range(n):
                c = (self.scan - back) % n
                if self.stats_used[c] and self.stats_done[c].query():
                    j = c
                    break
            else:
                return  # nothing newer has arrived: keep the layout
        else:
            self.stats_done[j].synchronize()
        rc = lib().sjq_dim_plan_end(self.carr, len(self.names), self.key_col, self.npay, ctypes.byref(self.opts),
                                    self.stats[j].data_ptr(), ctypes.byref(self.layout))
        if rc != 0:
            raise SjqError(rc, "sjq_dim_plan_end")
        self.planned = True

    def finish(self) -> Table:
        """Choose the layout (waiting for the scan unless reuse_layout allows an earlier one), enqueue the
        build on the side stream."""
        self._choose_layout()
        i = self.turn
        self.turn ^= 1
        main = torch.cuda.current_stream(self.device)
        if self.mems[i] is None or self.mems[i].numel() < self.layout.table_bytes:
            with torch.cuda.device(self.device):
                self.mems[i] = torch.empty(self.layout.table_bytes, dtype=torch.uint8, device=self.device)
            self.side.wait_stream(main)
        # The build overwrites buffer i, which the table returned two calls ago lives in: it must follow
        # whatever the current stream had queued by the time of the previous call (the runs on that table),
        # not the runs on the previous table, which read the other buffer.  A table is therefore valid for
        # work enqueued on the current stream before the next call of finish().
        if self.guard_set[i]:
            self.side.wait_event(self.guards[i])
        self.guards[i ^ 1].record(main)
        self.guard_set[i ^ 1] = True
        mem = self.mems[i]
        handle = ctypes.c_void_p()
        rc = lib().sjq_build_dim(self.carr, len(self.names), self.parr, self.npreds, self.key_col, self.pay,
                                 self.npay, ctypes.byref(self.layout), mem.data_ptr(), mem.numel(),
                                 self.status.data_ptr(), self.side.cuda_stream, ctypes.byref(handle))
        if rc != 0:
            raise SjqError(rc, "sjq_build_dim")
        layout = DimLayout.from_buffer_copy(self.layout)
        return Table(handle.value, layout, mem, self.status)


def workload_builders(w, dims: dict, reuse_layout: bool = False) -> dict:
    return {d.name: TableBuilder(dims[d.name], d.key, d.preds, d.payloads,
                                 force_kind=FORCE_HASH if d.force_hash else 0, reuse_layout=reuse_layout)
            for d in w.dims}


def build_tables(builders: dict) -> dict:
    """Plan all dimensions (one wait each, scans overlapping on side streams), build them concurrently,
    and make the current stream wait for the builds."""
    for b in builders.values():
        b.begin()
    tables = {name: b.finish() for name, b in builders.items()}
    for b in builders.values():
        torch.cuda.current_stream(b.device).wait_stream(b.side)
    return tables


def unfused_scratch(rows: int, njoins: int, device="cuda:0") -> torch.Tensor:
    """Scratch for RunOpts.unfused_scratch (the operator-at-a-time ablation): sjq_unfused_scratch_bytes."""
    n = ctypes.c_size_t(0)
    L = lib()
    L.sjq_unfused_scratch_bytes.restype = ctypes.c_int32
    L.sjq_unfused_scratch_bytes.argtypes = [ctypes.c_int64, ctypes.c_int, ctypes.POINTER(ctypes.c_size_t)]
    rc = L.sjq_unfused_scratch_bytes(rows, njoins, ctypes.byref(n))
    if rc != 0:
        raise SjqError(rc, "sjq_unfused_scratch_bytes")
    return torch.empty(n.value, dtype=torch.uint8, device=device)


def sample_preds(fact: dict, preds=()) -> tuple:
    """sjq_pred_sample: measured pass fraction (parts per million) of every fact predicate, in the form
    RunOpts.pass_ppm takes.  Synchronises the current stream."""
    if not preds:
        return ()
    names = list(fact.keys())
    tensors = [fact[n] for n in names]
    device = tensors[0].device
    with torch.cuda.device(device):
        carr = _cols(tensors)
        parr, keep = _preds(preds, names)
        scratch = torch.empty(PLAN_SCRATCH_BYTES, dtype=torch.uint8, device=device)
        out = (ctypes.c_int32 * len(preds))()
        rc = lib().sjq_pred_sample(carr, len(names), parr, len(preds), scratch.data_ptr(), _stream_ptr(device), out)
        if rc != 0:
            raise SjqError(rc, "sjq_pred_sample")
    return tuple(out)


class PredSampler:
    """The fact predicates of a query prepared for repeated sampling on a side stream (sjq_pred_sample_begin /
    _end), so that a planning step shares one wait between the dimension scans and the sample."""

    def __init__(self, fact: dict, preds=()):
        self.names = list(fact.keys())
        self.tensors = [fact[n] for n in self.names]
        self.device = self.tensors[0].device
        self.npreds = len(preds)
        with torch.cuda.device(self.device):
            self.carr = _cols(self.tensors)
            self.parr, self._keep = _preds(preds, self.names)
            self.scratch = torch.empty(PLAN_SCRATCH_BYTES, dtype=torch.uint8, device=self.device)
            self.counts = torch.zeros(MAX_PREDS + 1, dtype=torch.int64, pin_memory=True)
            self.side = torch.cuda.Stream(self.device)
        self.out = (ctypes.c_int32 * max(1, self.npreds))()

    def begin(self):
        if self.npreds:
            rc = lib().sjq_pred_sample_begin(self.carr, len(self.names), self.parr, self.npreds,
                                             self.scratch.data_ptr(), self.counts.data_ptr(), self.side.cuda_stream)
            if rc != 0:
                raise SjqError(rc, "sjq_pred_sample_begin")

    def end(self) -> tuple:
        if not self.npreds:
            return ()
        self.side.synchronize()
        rc = lib().sjq_pred_sample_end(self.counts.data_ptr(), self.npreds, self.out)
        if rc != 0:
            raise SjqError(rc, "sjq_pred_sample_end")
        return tuple(self.out[: self.npreds])


@dataclass
class Result:
    mode: str
    sums: torch.Tensor
    counts: Optional[torch.Tensor]
    keys: Optional[torch.Tensor]
    n_groups: Optional[torch.Tensor]
    status_dev: torch.Tensor
    workspace: Optional[torch.Tensor]
    info: RunInfo = field(default_factory=RunInfo)
    joined: Optional[torch.Tensor] = None  # SCALAR / DENSE: sums, counts and one spare cell as views of one int64
    #                                        buffer, so that a multi-GPU merge is a single all-reduce

    def status(self) -> int:
        return int(self.status_dev.item())

    def check(self) -> "Result":
        st = self.status()
        if st != 0:
            raise SjqError(st, "sjq_run")
        return self

    def sort(self) -> "Result":
        """sjq_result_sort: put a HASHED result into ascending key order, in place, on the current stream."""
        capacity = self.keys.numel()
        L = lib()
        L.sjq_result_sort_scratch_bytes.restype = ctypes.c_int32
        L.sjq_result_sort_scratch_bytes.argtypes = [ctypes.c_int64, ctypes.POINTER(ctypes.c_size_t)]
        L.sjq_result_sort.restype = ctypes.c_int32
        L.sjq_result_sort.argtypes = [ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p,
                                      ctypes.c_int64, ctypes.c_void_p, ctypes.c_size_t, ctypes.c_void_p]
        need = ctypes.c_size_t(0)
        rc = L.sjq_result_sort_scratch_bytes(capacity, ctypes.byref(need))
        if rc != 0:
            raise SjqError(rc, "sjq_result_sort_scratch_bytes")
        device = self.keys.device
        with torch.cuda.device(device):
            scratch = torch.empty(need.value, dtype=torch.uint8, device=device)
            rc = L.sjq_result_sort(self.keys.data_ptr(), self.sums.data_ptr(), self.counts.data_ptr(),
                                   self.n_groups.data_ptr(), capacity, scratch.data_ptr(), scratch.numel(),
                                   _stream_ptr(device))
        if rc != 0:
            raise SjqError(rc, "sjq_result_sort")
        return self

    def hashed_sorted(self):
        """(keys, sums, counts) of a HASHED result in ascending key order (copies; the result is left as it is)."""
        tmp = Result("HASHED", self.sums.clone(), self.counts.clone(), self.keys.clone(), self.n_groups,
                     self.status_dev, None).sort()
        n = int(self.n_groups.item())
        return tmp.keys[:n], tmp.sums[:n], tmp.counts[:n]


def _term(t, names) -> _Term:
    if t is None:
        return _Term(0, 0, 0, 0)
    if t.src == "FACT":
        return _Term(0, names.index(t.a), 0, t.mult)
    return _Term(1, int(t.a), t.b, t.mult)


def alloc_result(mode: str, num_groups: int, capacity: int, want_count: bool, device) -> Result:
    spec = _ResultSpec(MODES[mode], num_groups, capacity)
    n = 1 if mode == "SCALAR" else num_groups if mode == "DENSE" else capacity
    keys = n_groups = ws = joined = None
    if mode != "HASHED":
        # one allocation: [sums | counts | one cell for the merged status]; each part starts 16-byte aligned
        pad = (n + 1) // 2 * 2
        joined = torch.empty(2 * pad + 2 if want_count else pad + 2, dtype=torch.int64, device=device)
        sums = joined[:n]
        counts = joined[pad:pad + n] if want_count else None
    else:
        sums = torch.empty(n, dtype=torch.int64, device=device)
        counts = torch.empty(n, dtype=torch.int64, device=device)
    if mode == "HASHED":
        keys = torch.empty(n, dtype=torch.int64, device=device)
        n_groups = torch.zeros(1, dtype=torch.int64, device=device)
        nbytes = ctypes.c_size_t(0)
        rc = lib().sjq_run_workspace_bytes(ctypes.byref(spec), ctypes.byref(nbytes))
        if rc != 0:
            raise SjqError(rc, "sjq_run_workspace_bytes")
        ws = torch.empty(nbytes.value, dtype=torch.uint8, device=device)
    status = torch.zeros(1, dtype=torch.int32, device=device)
    return Result(mode, sums, counts, keys, n_groups, status, ws, joined=joined)


def merge_groups(keys: torch.Tensor, sums: torch.Tensor, counts: torch.Tensor, capacity: int,
                 result: Optional[Result] = None) -> Result:
    """sjq_merge_groups: fold lists of (key, sum, count) triples (CUDA int64 tensors of equal length) into
    a HASHED result with one entry per distinct key."""
    device = keys.device
    n = keys.numel()
    for t in (keys, sums, counts):
        if t.dtype != torch.int64 or not t.is_cuda or not t.is_contiguous() or t.numel() != n:
            raise ValueError("merge_groups takes contiguous int64 CUDA tensors of equal length")
    with torch.cuda.device(device):
        res = result if result is not None else alloc_result("HASHED", 0, capacity, True, device)
        cres = _result_struct(res)
        rc = lib().sjq_merge_groups(keys.data_ptr(), sums.data_ptr(), counts.data_ptr(), n, capacity,
                                    ctypes.byref(cres), _stream_ptr(device))
        if rc != 0:
            raise SjqError(rc, "sjq_merge_groups")
    return res


def _query(names: Sequence[str], preds, joins, key, agg):
    """Marshal the query part of a call: (predicates, joins, key expression or None, aggregate expression,
    objects that must outlive the call)."""
    parr, keep = _preds(preds, names)
    jarr = (_Join * max(1, len(joins)))()
    for j, (fk, table) in enumerate(joins):
        jarr[j] = _Join(names.index(fk), table.handle)
    kexpr = None
    if key is not None:
        if len(key.terms) > MAX_KEY_TERMS:
            raise ValueError("too many key terms")
        kexpr = _KeyExpr()
        for i, t in enumerate(key.terms):
            kexpr.t[i] = _term(t, names)
        kexpr.nterms, kexpr.offset, kexpr.modulo = len(key.terms), key.offset, key.modulo
    aexpr = _AggExpr(AGGS[agg.op], _term(agg.x, names), _term(agg.y, names), int(agg.want_count))
    return parr, jarr, kexpr, aexpr, keep


def _result_struct(res: "Result") -> _Result:
    return _Result(res.sums.data_ptr(), res.counts.data_ptr() if res.counts is not None else None,
                   res.keys.data_ptr() if res.keys is not None else None,
                   res.n_groups.data_ptr() if res.n_groups is not None else None, res.status_dev.data_ptr(),
                   res.workspace.data_ptr() if res.workspace is not None else None,
                   res.workspace.numel() if res.workspace is not None else 0)


def run(fact: dict, preds=(), joins=(), key=None, agg=None, mode: str = "SCALAR", num_groups: int = 1,
        capacity: int = 0, opts: Optional[RunOpts] = None, result: Optional[Result] = None) -> Result:
    """sjq_run over a dict of CUDA tensors.  joins: sequence of (fk column name, Table)."""
    names = list(fact.keys())
    tensors = [fact[n] for n in names]
    device = tensors[0].device
    with torch.cuda.device(device):
        carr = _cols(tensors)
        parr, jarr, kexpr, aexpr, keep = _query(names, preds, joins, key, agg)
        spec = _ResultSpec(MODES[mode], num_groups, capacity)
        res = result if result is not None else alloc_result(mode, num_groups, capacity, agg.want_count, device)
        cres = _result_struct(res)
        copts = (opts or RunOpts()).to_c()
        if not copts.hot_scratch and copts.hot_keys != 2 and any(t.layout.kind_name.startswith("HASH") for _, t in joins):
            scratch = _hot_scratch(device)  # one per device, reused by every run (runs on one stream are ordered)
            copts.hot_scratch, copts.hot_scratch_bytes = scratch.data_ptr(), scratch.numel()
        rc = lib().sjq_run(carr, len(names), parr, len(preds), jarr, len(joins),
                           ctypes.byref(kexpr) if kexpr is not None else None, ctypes.byref(aexpr),
                           ctypes.byref(spec), ctypes.byref(cres), ctypes.byref(copts), _stream_ptr(device),
                           ctypes.byref(res.info))
        if rc != 0:
            raise SjqError(rc, "sjq_run")
    return res


STATIC_MAX_GROUPS = 65536
HOT_SCRATCH_BYTES = 3 * 1048576 + 65536  # SJQ_HOT_SCRATCH_BYTES
_hot_scratch_by_device: dict = {}


def _hot_scratch(device) -> torch.Tensor:
    """Scratch for the hot-key table of open-addressing joins (sjq_run_opts.hot_scratch).  The library
    allocates nothing; this binding keeps one buffer per device.  Runs that may overlap on different streams
    need a buffer each: pass RunOpts.hot_scratch."""
    key = torch.device(device).index if torch.device(device).index is not None else torch.cuda.current_device()
    if key not in _hot_scratch_by_device:
        _hot_scratch_by_device[key] = torch.empty(HOT_SCRATCH_BYTES, dtype=torch.uint8, device=device)
    return _hot_scratch_by_device[key]


def run_hashed_static(fact: dict, preds=(), joins=(), key=None, agg=None, capacity: int = 0,
                      opts: Optional[RunOpts] = None, result: Optional[Result] = None) -> Result:
    """sjq_run_hashed_static: a hashed group-by whose group table is a fixed array inside the library,
    for callers that cannot allocate device memory.  The caller still supplies the result arrays
    (`result`, or fresh tensors here for convenience); no workspace is passed.  At most
    STATIC_MAX_GROUPS groups; calls must not overlap on the GPU because they share the one table."""
    names = list(fact.keys())
    tensors = [fact[n] for n in names]
    device = tensors[0].device
    with torch.cuda.device(device):
        carr = _cols(tensors)
        parr, jarr, kexpr, aexpr, keep = _query(names, preds, joins, key, agg)
        if result is None:
            n = max(1, capacity)
            result = Result("HASHED", torch.empty(n, dtype=torch.int64, device=device),
                            torch.empty(n, dtype=torch.int64, device=device),
                            torch.empty(n, dtype=torch.int64, device=device),
                            torch.zeros(1, dtype=torch.int64, device=device),
                            torch.zeros(1, dtype=torch.int32, device=device), None)
        cres = _Result(result.sums.data_ptr(), result.counts.data_ptr(), result.keys.data_ptr(),
                       result.n_groups.data_ptr(), result.status_dev.data_ptr(), None, 0)
        copts = (opts or RunOpts()).to_c()
        rc = lib().sjq_run_hashed_static(carr, len(names), parr, len(preds), jarr, len(joins), ctypes.byref(kexpr),
                                         ctypes.byref(aexpr), capacity, ctypes.byref(cres), ctypes.byref(copts),
                                         _stream_ptr(device), ctypes.byref(result.info))
        if rc != 0:
            raise SjqError(rc, "sjq_run_hashed_static")
    return result


@dataclass
class HostResult:
    """Pinned host copies of a result (filled when the stream has synchronised)."""
    sums: torch.Tensor
    counts: Optional[torch.Tensor]
    keys: Optional[torch.Tensor]
    n_groups: Optional[torch.Tensor]
    status: torch.Tensor


def staging_bytes(fact: dict, chunk_rows: int) -> int:
    per = 0
    for t in fact.values():
        per += (chunk_rows * t.element_size() + 255) // 256 * 256
    return 2 * per


def host_transfer_plan(fact: dict, preds=(), joins=(), key=None, agg=None, opts: Optional[RunOpts] = None) -> dict:
    """sjq_host_transfer_plan: for each host column, ("copy" | "in place" | "not transferred", estimated
    share of the rows it is first read for) as run_host would treat it."""
    names = list(fact.keys())
    tensors = [fact[n] for n in names]
    carr = (_Col * len(tensors))()
    for i, t in enumerate(tensors):
        carr[i] = _Col(t.data_ptr(), 1 if t.dtype == torch.int64 else 0, t.numel())
    parr, jarr, kexpr, aexpr, keep = _query(names, preds, joins, key, agg)
    copts = (opts or RunOpts()).to_c()
    how = (ctypes.c_int32 * len(names))()
    share = (ctypes.c_double * len(names))()
    L = lib()
    L.sjq_host_transfer_plan.restype = ctypes.c_int32
    rc = L.sjq_host_transfer_plan(carr, len(names), parr, len(preds), jarr, len(joins),
                                  ctypes.byref(kexpr) if kexpr is not None else None, ctypes.byref(aexpr),
                                  ctypes.byref(copts), how, share)
    if rc != 0:
        raise SjqError(rc, "sjq_host_transfer_plan")
    label = ("copy", "in place", "not transferred")
    return {n: (label[how[i]], share[i]) for i, n in enumerate(names)}


def run_host(fact: dict, staging: torch.Tensor, chunk_rows: int, preds=(), joins=(), key=None, agg=None,
             mode: str = "SCALAR", num_groups: int = 1, capacity: int = 0, opts: Optional[RunOpts] = None,
             result: Optional[Result] = None, host: Optional[HostResult] = None):
    """sjq_run_host: `fact` is a dict of HOST tensors (pinned for full speed), `staging` a CUDA uint8
    tensor of at least staging_bytes(fact, chunk_rows).  Returns (Result, HostResult); synchronise the
    current stream before reading the host copies."""
    names = list(fact.keys())
    tensors = [fact[n] for n in names]
    device = staging.device
    with torch.cuda.device(device):
        carr = (_Col * len(tensors))()
        for i, t in enumerate(tensors):
            if t.is_cuda or t.dtype not in (torch.int32, torch.int64) or not t.is_contiguous():
                raise ValueError("run_host takes contiguous int32/int64 host tensors")
            carr[i] = _Col(t.data_ptr(), 1 if t.dtype == torch.int64 else 0, t.numel())
        parr, jarr, kexpr, aexpr, keep = _query(names, preds, joins, key, agg)
        spec = _ResultSpec(MODES[mode], num_groups, capacity)
        res = result if result is not None else alloc_result(mode, num_groups, capacity, agg.want_count, device)
        if host is None:
            pin = dict(pin_memory=True)
            host = HostResult(torch.empty_like(res.sums, device="cpu", **pin),
                              torch.empty_like(res.counts, device="cpu", **pin) if res.counts is not None else None,
                              torch.empty_like(res.keys, device="cpu", **pin) if res.keys is not None else None,
                              torch.zeros(1, dtype=torch.int64, **pin) if res.n_groups is not None else None,
                              torch.zeros(1, dtype=torch.int32, **pin))
        cres = _result_struct(res)
        copts = (opts or RunOpts()).to_c()
        rc = lib().sjq_run_host(carr, len(names), parr, len(preds), jarr, len(joins),
                                ctypes.byref(kexpr) if kexpr is not None else None, ctypes.byref(aexpr),
                                ctypes.byref(spec), ctypes.byref(cres), ctypes.byref(copts), staging.data_ptr(),
                                staging.numel(), chunk_rows, host.sums.data_ptr(),
                                host.counts.data_ptr() if host.counts is not None else None,
                                host.keys.data_ptr() if host.keys is not None else None,
                                host.n_groups.data_ptr() if host.n_groups is not None else None,
                                host.status.data_ptr(), _stream_ptr(device))
        if rc != 0:
            raise SjqError(rc, "sjq_run_host")
    return res, host


def run_workload_host(w, fact: dict, tables: dict, staging: torch.Tensor, chunk_rows: int,
                      opts: Optional[RunOpts] = None, result=None, host=None):
    fact = {c.name: fact[c.name] for c in w.fact_cols}
    return run_host(fact, staging, chunk_rows, w.preds, [(fk, tables[dn]) for fk, dn in w.joins], w.key, w.agg,
                    w.mode, w.num_groups, w.capacity, opts, result, host)


def jit_log() -> str:
    """Compiler output of the most recent run-time compilation of the fused kernel."""
    L = lib()
    L.sjq_jit_log.restype = ctypes.c_size_t
    L.sjq_jit_log.argtypes = [ctypes.c_char_p, ctypes.c_size_t]
    n = L.sjq_jit_log(None, 0)
    buf = ctypes.create_string_buffer(int(n) + 1)
    L.sjq_jit_log(buf, len(buf))
    return buf.value.decode(errors="replace")


def build_launches(table: "Table") -> int:
    """Kernels enqueued by sjq_dim_plan + sjq_build_dim for this table: the plan's two (counter
    initialisation, and the scan unless the dimension is empty) and what the build reports."""
    L = lib()
    L.sjq_table_kernel_launches.restype = ctypes.c_int32
    L.sjq_table_kernel_launches.argtypes = [ctypes.c_void_p]
    return 1 + (1 if table.layout.dim_rows > 0 else 0) + int(L.sjq_table_kernel_launches(table.handle))


def release() -> int:
    """sjq_release: drop the library's per-thread streams and events, compiled modules and cached answers."""
    L = lib()
    L.sjq_release.restype = ctypes.c_int32
    return int(L.sjq_release())


def build_workload_tables(w, dims: dict) -> dict:
    """dims: dimension name -> dict of CUDA column tensors (a workload description's dims)."""
    out = {}
    for d in w.dims:
        out[d.name] = build_dim(dims[d.name], d.key, d.preds, d.payloads,
                                force_kind=FORCE_HASH if d.force_hash else 0)
    return out


def run_workload(w, fact: dict, tables: dict, opts: Optional[RunOpts] = None,
                 result: Optional[Result] = None, sample: bool = False) -> Result:
    """Run a workload description.  sample: measure the fact predicates' pass fractions first (one small
    kernel and a stream synchronisation) unless the options already carry measured ones."""
    fact = {c.name: fact[c.name] for c in w.fact_cols}
    if sample and w.preds and not (opts is not None and any(opts.pass_ppm)):
        opts = replace(opts) if opts is not None else RunOpts()
        opts.pass_ppm = sample_preds(fact, w.preds)
    return run(fact, w.preds, [(fk, tables[dn]) for fk, dn in w.joins], w.key, w.agg, w.mode, w.num_groups,
               w.capacity, opts, result)
