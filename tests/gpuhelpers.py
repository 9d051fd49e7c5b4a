"""GPU-side test helpers: run a workload through the C ABI and through the
oracle on the same inputs and compare element by element (bit-exact)."""
import numpy as np
import torch

import oracle
import paper_2607_07632_b200 as sjq


def to_dev(arrays, device="cuda:0"):
    return {k: torch.from_numpy(np.ascontiguousarray(v)).to(device) for k, v in arrays.items()}


def oracle_result(w, fact, host_dims, check=True):
    dims = oracle.build_dims(w, host_dims)
    return dims, oracle.run(w, fact, dims, check=check)


def compare(w, res, exp):
    """res: sjq.Result (device), exp: oracle dict."""
    if w.mode == "SCALAR":
        assert int(res.sums[0].item()) == exp["sum"], (int(res.sums[0].item()), exp["sum"])
        if res.counts is not None:
            assert int(res.counts[0].item()) == exp["count"]
    elif w.mode == "DENSE":
        assert np.array_equal(res.sums.cpu().numpy(), exp["sums"])
        if res.counts is not None:
            assert np.array_equal(res.counts.cpu().numpy(), exp["counts"])
    else:
        k, s, c = res.hashed_sorted()
        assert np.array_equal(k.cpu().numpy(), exp["keys"])
        assert np.array_equal(s.cpu().numpy(), exp["sums"])
        assert np.array_equal(c.cpu().numpy(), exp["counts"])


def run_both(w, fact, host_dims, opts=None, check=True, dev_fact=None, tables=None):
    dims, exp = oracle_result(w, fact, host_dims, check=check)
    if tables is None:
        tables = sjq.build_workload_tables(w, {k: to_dev(v) for k, v in host_dims.items()})
        for t in tables.values():
            t.check()
    if dev_fact is None:
        dev_fact = to_dev(fact)
    res = sjq.run_workload(w, dev_fact, tables, opts)
    torch.cuda.synchronize()
    return res, exp, tables
