"""CPU-only checks of the boundary: the C-ABI library loads and exports every
symbol the public header declares, and host-side argument validation answers
without a GPU (no compute is attempted)."""
import ctypes
import os
import re

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


@pytest.fixture(scope="module")
def libsjq():
    from paper_2607_07632_b200 import build

    return ctypes.CDLL(build.build())


def _declared_symbols():
    names = set()
    for fn in os.listdir(os.path.join(ROOT, "include")):
        text = open(os.path.join(ROOT, "include", fn)).read()
        text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
        names |= set(re.findall(r"\b(sjq_[a-z0-9_]+)\s*\(", text))
    return names


def test_library_exports_every_declared_symbol(libsjq):
    names = _declared_symbols()
    assert {"sjq_dim_plan", "sjq_build_dim", "sjq_run", "sjq_table_info", "sjq_table_destroy",
            "sjq_run_workspace_bytes", "sjq_strerror", "sjq_version"} <= names
    for n in names:
        assert hasattr(libsjq, n), n


def test_strerror_and_workspace_size(libsjq):
    import paper_2607_07632_b200.sjq as b

    assert b.strerror(0) == "ok" and "duplicate" in b.strerror(16)
    spec = b._ResultSpec(b.MODES["HASHED"], 0, 1000)
    n = ctypes.c_size_t(0)
    assert b.lib().sjq_run_workspace_bytes(ctypes.byref(spec), ctypes.byref(n)) == 0
    # 2048 slots + the side slot, three int64 arrays
    assert 3 * 2049 * 8 <= n.value <= 3 * 2049 * 8 + 3 * 256
    spec = b._ResultSpec(b.MODES["DENSE"], 7000, 0)
    assert b.lib().sjq_run_workspace_bytes(ctypes.byref(spec), ctypes.byref(n)) == 0 and n.value == 0
    spec = b._ResultSpec(b.MODES["HASHED"], 0, 0)
    assert b.lib().sjq_run_workspace_bytes(ctypes.byref(spec), ctypes.byref(n)) == 1


def test_null_arguments_rejected_without_gpu(libsjq):
    import paper_2607_07632_b200.sjq as b

    assert b.lib().sjq_run(None, 0, None, 0, None, 0, None, None, None, None, None, None, None) == 1
    assert b.lib().sjq_dim_plan(None, 0, None, 0, 0, None, 0, None, None, None, None) == 1
    assert b.lib().sjq_table_info(None, None) == 1
    b.lib().sjq_table_destroy(None)


def test_product_never_imports_the_oracle():
    pkg = os.path.join(ROOT, "paper_2607_07632_b200")
    for dirpath, _, files in os.walk(pkg):
        for f in files:
            if f.endswith((".py", ".cu", ".cuh", ".h")):
                text = open(os.path.join(dirpath, f)).read()
                assert "oracle" not in text.lower(), f


def test_device_source_compiles_for_builtin_query_shapes(libsjq):
    """Run-time specialisation needs no device to compile: every built-in query shape (scalar with a
    product aggregate, four joins with a shared-memory group table, 64-bit open addressing with a
    presence bitmap, no queues with a global group hash table) must compile for sm_100a with NVRTC."""
    libsjq.sjq_jit_selftest.restype = ctypes.c_int32
    libsjq.sjq_jit_selftest.argtypes = [ctypes.c_int32, ctypes.c_char_p, ctypes.c_size_t]
    n = libsjq.sjq_jit_selftest(-1, None, 0)
    assert n >= 4
    for i in range(n):
        log = ctypes.create_string_buffer(1 << 16)
        rc = libsjq.sjq_jit_selftest(i, log, len(log))
        assert rc == 0, (i, log.value.decode()[:2000])
    assert libsjq.sjq_jit_selftest(n, None, 0) == 1  # no such shape: invalid argument


def test_release_without_a_device_is_harmless(libsjq):
    libsjq.sjq_release.restype = ctypes.c_int32
    assert libsjq.sjq_release() >= 0
    assert libsjq.sjq_release() == 0  # nothing left to give back
    assert libsjq.sjq_table_kernel_launches(None) == 0


def test_build_rejects_inconsistent_layouts_on_the_host(libsjq):
    """sjq_build_dim takes the table shape from its caller.  Every size it uses is recomputed from the shape
    fields, so a layout whose fields contradict one another (or whose table_bytes was not recomputed after
    an edit) is rejected before anything is enqueued: no device is needed to see that, and the pointers
    below are never dereferenced."""
    import paper_2607_07632_b200.sjq as b

    n = 1000
    cols = (b._Col * 2)(b._Col(0x10000, 0, n), b._Col(0x20000, 0, n))
    pay = (ctypes.c_int * 1)(1)
    handle = ctypes.c_void_p()

    def build(layout, table_bytes=1 << 30):
        return b.lib().sjq_build_dim(cols, 2, None, 0, 0, pay, 1, ctypes.byref(layout), 0x100000, table_bytes,
                                     0x30000, None, ctypes.byref(handle))

    def direct():
        L = b.DimLayout()
        L.kind, L.key_dtype, L.npayload, L.code_bits = 2, 0, 1, 8  # DIRECT_U8
        L.dim_rows, L.entries, L.kmin, L.kmax, L.slots = n, n, 1, n, n
        L.pay_bits[0] = 3
        L.filter_bits = 1152
        L.table_bytes = b.layout_bytes(L)
        return L

    def hashed():
        L = direct()
        L.kind, L.code_bits, L.slots, L.filter_bits = 6, 32, 2048, 16384  # HASH_I32
        L.table_bytes = b.layout_bytes(L)
        return L

    for mk in (direct, hashed):
        good = mk()
        assert good.table_bytes > good.slots
        assert build(good, good.table_bytes - 1) == 5  # consistent, but the caller's buffer is too small
        L = mk()
        L.table_bytes -= 256  # stale size
        assert build(L) == 1
        L = mk()
        L.code_bits = 16  # does not match the kind
        assert build(L) == 1
        L = mk()
        L.slots = 0
        assert build(L) == 1
        L = mk()
        L.dim_rows = n + 1  # planned for another dimension
        assert build(L) == 1
    L = hashed()
    L.slots = 2046  # an open-addressing table is made of whole buckets
    with pytest.raises(b.SjqError):
        b.layout_bytes(L)
    L.table_bytes = hashed().table_bytes
    assert build(L) == 1
    L = hashed()
    L.filter_bits = 1000  # the presence bitmap of an open-addressing table is a power of two
    assert build(L) == 1
    L = direct()
    L.filter_bits = 640  # fewer bits than slots
    assert build(L) == 1
    L = direct()
    L.kind, L.code_bits = 1, 0  # a bitmap table cannot carry the payload the call names
    assert build(L) == 1


def test_mis_guessed_predicates_do_not_send_dense_columns_over_the_bus_piecemeal(libsjq):
    """sjq_run_host reads a column in place over the bus when the planner expects only a few per cent of the
    rows to reach it.  By their operators alone two equality predicates look as if they kept 1 % of the rows;
    here they keep all of them.  The planning call measures predicates on host-resident columns, so every
    column must be planned as a whole copy (and with predicates that keep nothing, later columns are expected
    to be reached by almost no row)."""
    import torch

    import paper_2607_07632_b200.sjq as b
    from datagen.workloads import AggExpr, Pred, Term

    n = 100_000
    fact = {"a": torch.full((n,), 7, dtype=torch.int32), "b": torch.full((n,), 9, dtype=torch.int64),
            "m": torch.arange(n, dtype=torch.int32), "unused": torch.zeros(n, dtype=torch.int32)}
    agg = AggExpr("COL", Term("FACT", "m"))
    plan = b.host_transfer_plan(fact, (Pred("a", "EQ", 7), Pred("b", "EQ", 9)), (), None, agg)
    assert plan["unused"][0] == "not transferred"
    for c in ("a", "b", "m"):
        assert plan[c] == ("copy", 1.0), (c, plan[c])
    # the same predicates keeping nothing: the measured share of rows reaching the later columns is tiny
    plan = b.host_transfer_plan(fact, (Pred("a", "EQ", 8), Pred("b", "EQ", 9)), (), None, agg)
    assert plan["a"][1] == 1.0 and plan["m"][1] < 1e-4
    # a caller's own measured fractions are taken as they are
    plan = b.host_transfer_plan(fact, (Pred("a", "EQ", 8), Pred("b", "EQ", 9)), (), None, agg,
                                b.RunOpts(pass_ppm=(500_000, 500_000)))
    assert abs(plan["m"][1] - 0.25) < 1e-9


def test_sampled_counters_become_parts_per_million(libsjq):
    import paper_2607_07632_b200.sjq as b

    counts = (ctypes.c_int64 * 17)(*([262144, 0, 26, 262144, 131072] + [0] * 12))
    out = (ctypes.c_int32 * 4)()
    assert b.lib().sjq_pred_sample_end(counts, 4, out) == 0
    assert list(out) == [1, 99, 1_000_000, 500_000]  # none seen -> 1 ppm, never "unknown"
    assert b.lib().sjq_pred_sample_end(None, 4, out) == 1
