"""Row-sharded execution over several GPUs (one process per GPU).

The fact table is cut into contiguous row ranges, one per rank; every rank
holds a replica of the (small) dimension tables and runs the unchanged
single-GPU pipeline on its range.  Because integer sums are exact and
commutative, adding the per-rank results gives the whole-table result: a
scalar or dense result takes ONE all-reduce over a buffer that joins sums,
counts and the status words (8 or 16 bytes per group), a hashed result one
all-gather of the per-rank (key, sum, count) lists followed by a merge of
equal keys (sjq_merge_groups on the GPU).  No probe ever reads another GPU's
memory.  Only `torch.distributed` plumbing lives here; it works the same over
NCCL (GPU tensors) and gloo (CPU tensors, with the merge step supplied by the
caller).
"""
from __future__ import annotations

import torch
import torch.distributed as dist

# Device-detected status codes are 16 .. 21; the joined buffer carries, per code, how many ranks reported it
# (8 bits each), so that one SUM all-reduce also merges the status words.
_STATUS_BASE, _STATUS_CODES = 16, 6


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


def rank_rows(rank: int, world: int, n: int, scaling: str = "weak") -> tuple[int, int]:
    """(first row, row count) of `rank` in the global row space.  "weak": every rank owns its own n rows
    (rows rank*n ..), the table grows with the ranks; "strong": one table of n rows cut by shard_rows."""
    if scaling == "weak":
        if world <= 0 or not (0 <= rank < world) or n < 0:
            raise ValueError("bad shard request")
        return rank * n, n
    if scaling == "strong":
        b, e = shard_rows(rank, world, n)
        return b, e - b
    raise ValueError("scaling is 'weak' or 'strong'")


def _status_flags(status: torch.Tensor) -> torch.Tensor:
    """int64 word with the count field of this rank's status code set to one (zero when the status is 0)."""
    s = status.to(torch.int64).reshape(())
    slot = torch.clamp(s - _STATUS_BASE, 0, _STATUS_CODES - 1)
    return torch.where(s != 0, torch.ones_like(s) << (8 * slot), torch.zeros_like(s))


def _merged_status(flags: torch.Tensor) -> torch.Tensor:
    """The lowest status code any rank reported (0 if none), as int32[1]."""
    f = flags.reshape(())
    code = torch.zeros_like(f)
    for slot in reversed(range(_STATUS_CODES)):
        code = torch.where(((f >> (8 * slot)) & 0xFF) != 0, torch.full_like(f, _STATUS_BASE + slot), code)
    return code.to(torch.int32).reshape(1)


def merge_dense(sums: torch.Tensor, counts: torch.Tensor | None, status: torch.Tensor | None = None,
                joined: torch.Tensor | None = None, group=None):
    """In-place sum over ranks of a scalar or dense result with a single all-reduce; the status word becomes
    the lowest code any rank reported.  `joined`: a buffer of which `sums` and `counts` are views and whose last
    cell is spare (what alloc_result provides): it is reduced in place, without a copy; otherwise the parts are
    joined into a temporary and copied back."""
    flags = _status_flags(status) if status is not None else None
    if joined is not None:
        joined[-1] = flags if flags is not None else 0
        dist.all_reduce(joined, op=dist.ReduceOp.SUM, group=group)
        merged = joined[-1]
    else:
        parts = [sums.reshape(-1)] + ([counts.reshape(-1)] if counts is not None else [])
        tail = flags.reshape(1) if flags is not None else torch.zeros(1, dtype=torch.int64, device=sums.device)
        buf = torch.cat(parts + [tail])
        dist.all_reduce(buf, op=dist.ReduceOp.SUM, group=group)
        n = sums.numel()
        sums.copy_(buf[:n].reshape(sums.shape))
        if counts is not None:
            counts.copy_(buf[n:2 * n].reshape(counts.shape))
        merged = buf[-1]
    if status is not None:
        status.copy_(_merged_status(merged).reshape(status.shape))
    return sums, counts


def _combine_on_gpu(capacity: int):
    def combine(keys, sums, counts):
        from . import sjq

        res = sjq.merge_groups(keys, sums, counts, capacity)
        return res.keys, res.sums, res.counts, res.n_groups, res.status_dev

    return combine


def merge_hashed(keys: torch.Tensor, sums: torch.Tensor, counts: torch.Tensor, n_groups, capacity: int | None = None,
                 status: torch.Tensor | None = None, combine=None, group=None):
    """All-gather the per-rank (key, sum, count) lists (two collectives: the list lengths, then one padded
    buffer holding all three arrays) and merge equal keys.  `combine(keys, sums, counts)` folds the gathered
    triples and returns (keys, sums, counts, n_groups, status); by default it is the library's merge kernel
    (CUDA tensors only; `capacity` bounds the number of distinct keys, default: the sum of the list lengths).
    Returns (keys[:n], sums[:n], counts[:n]) in no particular order, the same set on every rank; `status`, if
    given, receives the worst of the per-rank words and the merge's own."""
    world = dist.get_world_size(group)
    dev = keys.device
    n_mine = int(n_groups.item()) if torch.is_tensor(n_groups) else int(n_groups)
    head = torch.zeros(2, dtype=torch.int64, device=dev)
    head[0] = n_mine
    if status is not None:
        head[1] = _status_flags(status)
    heads = [torch.zeros_like(head) for _ in range(world)]
    dist.all_gather(heads, head, group=group)
    sizes = [int(h[0].item()) for h in heads]
    flags = sum(h[1] for h in heads)
    cap = max(max(sizes), 1)
    pad = torch.zeros(3, cap, dtype=torch.int64, device=dev)
    pad[0, :n_mine], pad[1, :n_mine], pad[2, :n_mine] = keys[:n_mine], sums[:n_mine], counts[:n_mine]
    out = [torch.empty_like(pad) for _ in range(world)]
    dist.all_gather(out, pad, group=group)
    k = torch.cat([o[0, :s] for o, s in zip(out, sizes)])
    s = torch.cat([o[1, :s] for o, s in zip(out, sizes)])
    c = torch.cat([o[2, :s] for o, s in zip(out, sizes)])
    if combine is None:
        if not k.is_cuda:
            raise ValueError("merging on the CPU needs a `combine` function: the library's merge is a CUDA kernel")
        combine = _combine_on_gpu(capacity if capacity else max(sum(sizes), 1))
    mk, ms, mc, mn, mstatus = combine(k, s, c)
    n = int(mn.item()) if torch.is_tensor(mn) else int(mn)
    if status is not None:
        worst = _merged_status(flags)
        own = mstatus.to(torch.int32).reshape(1) if mstatus is not None else torch.zeros_like(worst)
        status.copy_(torch.where(worst != 0, worst, own.to(worst.device)).reshape(status.shape))
    return mk[:n], ms[:n], mc[:n]


def merge_result(res, combine=None, group=None):
    """The exchange step of one row-sharded query, for every result mode: `res` is this rank's result
    (an object with mode, sums, counts, keys, n_groups, status_dev and optionally joined, like the binding's
    Result).  SCALAR / DENSE: reduced in place, returns (sums, counts).  HASHED: returns the merged
    (keys, sums, counts) lists; `res` itself keeps this rank's part."""
    if res.mode == "HASHED":
        return merge_hashed(res.keys, res.sums, res.counts, res.n_groups, capacity=res.keys.numel(),
                            status=res.status_dev, combine=combine, group=group)
    return merge_dense(res.sums, res.counts, res.status_dev, joined=getattr(res, "joined", None), group=group)
