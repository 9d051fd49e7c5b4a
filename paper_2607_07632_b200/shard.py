"""Row-sharded execution over several GPUs (one process per GPU).

The fact table is cut into contiguous row ranges, one per rank; every rank
holds a replica of the (small) dimension tables and runs the unchanged
single-GPU pipeline on its range.  Because integer sums are exact and
commutative, adding the per-rank results gives the whole-table result: dense
and scalar results take one all-reduce (8 bytes per group), hashed results an
all-gather of the per-rank (key, sum, count) lists followed by a merge.  No
probe ever reads another GPU's memory.  Only `torch.distributed` plumbing lives
here; it works the same over NCCL (GPU tensors) and gloo (CPU tensors).
"""
from __future__ import annotations

import torch
import torch.distributed as dist


def shard_rows(rank: int, world: int, n: int) -> tuple[int, int]:
    """Contiguous row range [begin, end) of `rank`; ranges differ by at most 4 rows and start on a
    multiple of 4 so that every shard's columns stay 16-byte aligned."""
    if world <= 0 or not (0 <= rank < world) or n < 0:
        raise ValueError("bad shard request")
    quads = (n + 3) // 4
    base, extra = divmod(quads, world)
    begin = 4 * (rank * base + min(rank, extra))
    end = 4 * ((rank + 1) * base + min(rank + 1, extra))
    return min(begin, n), min(end, n)


def merge_dense(sums: torch.Tensor, counts: torch.Tensor | None, status: torch.Tensor | None = None, group=None):
    """In-place sum over ranks of a scalar or dense result; the status word becomes the maximum."""
    dist.all_reduce(sums, op=dist.ReduceOp.SUM, group=group)
    if counts is not None:
        dist.all_reduce(counts, op=dist.ReduceOp.SUM, group=group)
    if status is not None:
        dist.all_reduce(status, op=dist.ReduceOp.MAX, group=group)
    return sums, counts


def merge_hashed(keys: torch.Tensor, sums: torch.Tensor, counts: torch.Tensor, n_groups: int, group=None):
    """All-gather the per-rank (key, sum, count) lists and merge equal keys.
    Returns (keys, sums, counts) in ascending key order, identical on every rank."""
    world = dist.get_world_size(group)
    n = torch.tensor([n_groups], dtype=torch.int64, device=keys.device)
    sizes = [torch.zeros_like(n) for _ in range(world)]
    dist.all_gather(sizes, n, group=group)
    sizes = [int(s.item()) for s in sizes]
    cap = max(max(sizes), 1)

    def gather(t):
        pad = torch.zeros(cap, dtype=t.dtype, device=t.device)
        pad[:n_groups] = t[:n_groups]
        out = [torch.empty_like(pad) for _ in range(world)]
        dist.all_gather(out, pad, group=group)
        return torch.cat([o[:s] for o, s in zip(out, sizes)])

    k, s, c = gather(keys), gather(sums), gather(counts)
    uk, inv = torch.unique(k, sorted=True, return_inverse=True)
    us = torch.zeros(uk.numel(), dtype=torch.int64, device=k.device).index_add_(0, inv, s)
    uc = torch.zeros(uk.numel(), dtype=torch.int64, device=k.device).index_add_(0, inv, c)
    return uk, us, uc
