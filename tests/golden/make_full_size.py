#!/usr/bin/env python
"""Writes the expected results of the five benchmark configurations at their
full sizes (tests/golden/full_*.json).  Calls only the CPU oracle and the
seeded input generator; nothing here touches the CUDA path.

    python tests/golden/make_full_size.py [c1 c2 c3 c5 c4:<sel>:<groups> city_pair ...]   (default: everything)

A dense result is stored whole (beyond 20 000 groups: its totals and a SHA-256
over the sums array followed by the counts array); a hashed result is stored as its group count,
the totals, and a SHA-256 over the (key, sum, count) triples in ascending key
order (int64 little-endian), which is what the GPU test recomputes.
"""
import hashlib
import json
import os
import sys
import time

import numpy as np

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
sys.path.insert(0, ROOT)

import oracle  # noqa: E402
from datagen import workloads as W  # noqa: E402


def triples_digest(keys, sums, counts):
    h = hashlib.sha256()
    h.update(np.ascontiguousarray(keys, dtype="<i8").tobytes())
    h.update(np.ascontiguousarray(sums, dtype="<i8").tobytes())
    h.update(np.ascontiguousarray(counts, dtype="<i8").tobytes())
    return h.hexdigest()


def compute(w, tag):
    t0 = time.time()
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    dims = oracle.build_dims(w, hd)
    # stream the fact table in slices so that no more than a few GB are resident
    step = 100_000_000
    acc = None
    for r0 in range(0, w.n_rows, step):
        n = min(step, w.n_rows - r0)
        fact = W.host_fact(w, r0, n)
        r = oracle.run(w, fact, dims)
        if w.mode == "SCALAR":
            part = {0: (r["sum"], r["count"])} if r["count"] else {}
        elif w.mode == "DENSE":
            part = (r["sums"], r["counts"])
        else:
            part = dict(zip(r["keys"].tolist(), zip(r["sums"].tolist(), r["counts"].tolist())))
        if acc is None:
            acc = part
        elif w.mode == "DENSE":
            acc = (acc[0] + part[0], acc[1] + part[1])
        else:
            for k, (s, c) in part.items():
                s0, c0 = acc.get(k, (0, 0))
                acc[k] = (s0 + s, c0 + c)
        del fact
    out = {"citation": "expected result of benchmark configuration '%s' at full size, written by "
                       "tests/golden/make_full_size.py from the CPU oracle (oracle/sjq_oracle.cpp) on the seeded "
                       "synthetic inputs of datagen/; slices of 100 M rows are added, which the split-and-add "
                       "invariant pinned in tests/test_oracle_pins.py makes exact" % w.name,
           "workload": w.name, "rows": w.n_rows, "mode": w.mode, "seed": w.seed,
           "dim_entries": {k: d.entries for k, d in dims.items()}}
    if w.mode == "SCALAR":
        s, c = acc.get(0, (0, 0))
        out.update(sum=int(s), count=int(c))
    elif w.mode == "DENSE" and w.num_groups > 20_000:
        # a large dense result is stored like a hashed one: totals and a digest of the two whole arrays
        h = hashlib.sha256()
        h.update(np.ascontiguousarray(acc[0], dtype="<i8").tobytes())
        h.update(np.ascontiguousarray(acc[1], dtype="<i8").tobytes())
        out.update(groups=int(np.count_nonzero(acc[1])), total_sum=int(acc[0].sum()), total_count=int(acc[1].sum()),
                   dense_sha256=h.hexdigest())
    elif w.mode == "DENSE":
        out.update(sums=[int(x) for x in acc[0]], counts=[int(x) for x in acc[1]])
    else:
        keys = np.array(sorted(acc), dtype=np.int64)
        sums = np.array([acc[k][0] for k in keys.tolist()], dtype=np.int64)
        counts = np.array([acc[k][1] for k in keys.tolist()], dtype=np.int64)
        out.update(groups=int(keys.size), total_sum=int(sums.sum()), total_count=int(counts.sum()),
                   sha256=triples_digest(keys, sums, counts), first_keys=keys[:4].tolist(),
                   first_sums=sums[:4].tolist(), first_counts=counts[:4].tolist())
    out["oracle_seconds"] = round(time.time() - t0, 1)
    with open(os.path.join(HERE, f"full_{tag}.json"), "w") as f:
        json.dump(out, f)
        f.write("\n")
    print(tag, "done in", out["oracle_seconds"], "s", flush=True)


def main():
    todo = sys.argv[1:] or (["c1", "c2", "c3", "c5"] + list(W.EXTRA_SHAPES) +
                            [f"c4:{s:g}:{g}" for s in W.C4_THRESHOLDS for g in W.C4_GROUPS])
    for item in todo:
        if item in W.EXTRA_SHAPES:
            w = W.EXTRA_SHAPES[item]()
            tag = item
        elif item.startswith("c4"):
            _, s, g = item.split(":")
            w = W.config4(600_000_000, float(s), int(g))
            tag = f"c4_s{float(s):g}_g{int(g)}"
        else:
            w = W.CONFIGS[item]()
            tag = item
        if os.path.exists(os.path.join(HERE, f"full_{tag}.json")):
            continue
        compute(w, tag)


if __name__ == "__main__":
    main()
