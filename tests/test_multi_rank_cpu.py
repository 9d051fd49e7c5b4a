"""The N > 1 path on CPU: two gloo ranks each evaluate their row shard (with
the oracle standing in for the per-rank GPU run) and merge through the
package's shard helpers; the merged result must equal the whole-table result."""
import os
import socket
import sys
from types import SimpleNamespace

import numpy as np
import pytest
import torch
import torch.distributed as dist
import torch.multiprocessing as mp

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))


def _free_port():
    with socket.socket() as s:
        s.bind(("127.0.0.1", 0))
        return s.getsockname()[1]


def _combine_cpu(keys, sums, counts):
    """Stand-in for the merge kernel (CUDA only) on CPU tensors: fold equal keys."""
    uk, inv = torch.unique(keys, return_inverse=True)
    us = torch.zeros(uk.numel(), dtype=torch.int64).index_add_(0, inv, sums)
    uc = torch.zeros(uk.numel(), dtype=torch.int64).index_add_(0, inv, counts)
    return uk, us, uc, uk.numel(), None


def _worker(rank, world, port, which, out_dir):
    sys.path.insert(0, ROOT)
    os.environ["MASTER_ADDR"] = "127.0.0.1"
    os.environ["MASTER_PORT"] = str(port)
    dist.init_process_group("gloo", rank=rank, world_size=world)
    try:
        import oracle
        from datagen import workloads as W
        from paper_2607_07632_b200 import shard

        w = {"dense": lambda: W.config3(200_003), "scalar": lambda: W.config1(100_001),
             "hashed": lambda: W.config4(120_001, 0.5, 100000, dim_rows=20000)}[which]()
        hd = {d.name: W.host_dim(w, d) for d in w.dims}
        dims = oracle.build_dims(w, hd)
        row0, rows = shard.rank_rows(rank, world, w.n_rows, "strong")
        fact = W.host_fact(w, row0, rows)
        part = oracle.run(w, fact, dims)
        # this rank's result in the shape the binding's Result has; one rank reports a device-side status
        st = torch.tensor([19 if (rank == 1 and which == "hashed") else 18 if (rank == 0 and which == "dense") else 0],
                          dtype=torch.int32)
        if w.mode == "HASHED":
            k, s, c = (torch.from_numpy(part[x].copy()) for x in ("keys", "sums", "counts"))
            res = SimpleNamespace(mode="HASHED", keys=k, sums=s, counts=c, n_groups=torch.tensor([k.numel()]),
                                  status_dev=st)
            uk, us, uc = shard.merge_result(res, combine=_combine_cpu)
            order = torch.argsort(uk)
            got = {"keys": uk[order].numpy(), "sums": us[order].numpy(), "counts": uc[order].numpy()}
        else:
            if w.mode == "SCALAR":
                s, c = torch.tensor([part["sum"]]), torch.tensor([part["count"]])
                res = SimpleNamespace(mode="SCALAR", sums=s, counts=c, status_dev=st)  # no joined buffer: copies
            else:
                n = part["sums"].size
                pad = (n + 1) // 2 * 2
                joined = torch.zeros(2 * pad + 2, dtype=torch.int64)  # the layout alloc_result gives a dense result
                s, c = joined[:n], joined[pad:pad + n]
                s.copy_(torch.from_numpy(part["sums"]))
                c.copy_(torch.from_numpy(part["counts"]))
                res = SimpleNamespace(mode="DENSE", sums=s, counts=c, status_dev=st, joined=joined)
            shard.merge_result(res)
            got = {"sums": s.numpy(), "counts": c.numpy()}
        got["status"] = st.numpy()
        np.savez(os.path.join(out_dir, f"r{rank}.npz"), **got)
    finally:
        dist.destroy_process_group()


@pytest.mark.parametrize("which", ["dense", "scalar", "hashed"])
def test_two_rank_shard_and_merge(which, tmp_path):
    import oracle
    from datagen import workloads as W

    mp.spawn(_worker, args=(2, _free_port(), which, str(tmp_path)), nprocs=2, join=True)
    w = {"dense": lambda: W.config3(200_003), "scalar": lambda: W.config1(100_001),
         "hashed": lambda: W.config4(120_001, 0.5, 100000, dim_rows=20000)}[which]()
    hd = {d.name: W.host_dim(w, d) for d in w.dims}
    whole = oracle.run(w, W.host_fact(w), oracle.build_dims(w, hd))
    for r in range(2):
        got = np.load(os.path.join(str(tmp_path), f"r{r}.npz"))
        # every rank ends with the same status word: the lowest code any rank reported
        assert int(got["status"][0]) == {"dense": 18, "scalar": 0, "hashed": 19}[which]
        if which == "scalar":
            assert int(got["sums"][0]) == whole["sum"] and int(got["counts"][0]) == whole["count"]
        else:
            for k in got.files:
                if k != "status":
                    assert np.array_equal(got[k], whole[k]), (which, k)


def test_shard_rows_cover_the_table_once():
    from paper_2607_07632_b200 import shard

    for n in (0, 1, 3, 4, 5, 1001, 600_000_000):
        for world in (1, 2, 3, 8):
            edges = [shard.shard_rows(r, world, n) for r in range(world)]
            assert edges[0][0] == 0 and edges[-1][1] == n
            for (b0, e0), (b1, e1) in zip(edges, edges[1:]):
                assert e0 == b1 and b0 <= e0
            assert all(b % 4 == 0 or b == n for b, _ in edges)


def test_rank_rows_weak_and_strong():
    from paper_2607_07632_b200 import shard

    assert [shard.rank_rows(r, 4, 1000, "weak") for r in range(4)] == [(0, 1000), (1000, 1000), (2000, 1000),
                                                                        (3000, 1000)]
    parts = [shard.rank_rows(r, 3, 1_200_000_001, "strong") for r in range(3)]
    assert parts[0][0] == 0 and sum(n for _, n in parts) == 1_200_000_001
    assert all(a + n == b for (a, n), (b, _) in zip(parts, parts[1:]))
    with pytest.raises(ValueError):
        shard.rank_rows(0, 2, 10, "other")
