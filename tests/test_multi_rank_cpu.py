"""The N > 1 path on CPU: two gloo ranks each evaluate their row shard (with
the oracle standing in for the per-rank GPU run) and merge through the
package's shard helpers; the merged result must equal the whole-table result."""
import os
import socket
import sys

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
        b, e = shard.shard_rows(rank, world, w.n_rows)
        fact = W.host_fact(w, b, e - b)
        part = oracle.run(w, fact, dims)
        if w.mode == "HASHED":
            k, s, c = (torch.from_numpy(part[x].copy()) for x in ("keys", "sums", "counts"))
            uk, us, uc = shard.merge_hashed(k, s, c, k.numel())
            got = {"keys": uk.numpy(), "sums": us.numpy(), "counts": uc.numpy()}
        else:
            if w.mode == "SCALAR":
                s, c = torch.tensor([part["sum"]]), torch.tensor([part["count"]])
            else:
                s, c = torch.from_numpy(part["sums"].copy()), torch.from_numpy(part["counts"].copy())
            st = torch.zeros(1, dtype=torch.int32)
            shard.merge_dense(s, c, st)
            got = {"sums": s.numpy(), "counts": c.numpy()}
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
        if which == "scalar":
            assert int(got["sums"][0]) == whole["sum"] and int(got["counts"][0]) == whole["count"]
        else:
            for k in got.files:
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
