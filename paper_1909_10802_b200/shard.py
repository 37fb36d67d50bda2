"""Splitting the parameter vector over ranks.

Every step of the master update is independent per parameter (Section 5.3 of the paper), so a
rank that holds a contiguous range of theta, v, m, of every saved copy and of every gradient
needs nothing from the other ranks: there is no exchange step and no collective on the data
path. Only the (tiny, host-side) arrival schedule is replicated.
"""
import hashlib

ALIGN = 32   # floats: shard boundaries fall on 128-byte boundaries


def shard_range(d, rank, world, align=ALIGN):
    """(j0, n): the contiguous range [j0, j0+n) of a d-vector owned by `rank`. Ranges tile
    [0, d) exactly, differ by at most `align` elements, and start on multiples of `align`."""
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    blocks = (d + align - 1) // align
    lo = (blocks * rank) // world * align
    hi = (blocks * (rank + 1)) // world * align
    lo, hi = min(lo, d), min(hi, d)
    return lo, hi - lo


def schedule_digest(schedule):
    """Digest of an arrival schedule; ranks compare digests before running."""
    return hashlib.sha256(",".join(map(str, schedule)).encode()).hexdigest()


def assert_same_schedule(schedule, dist):
    """All ranks of the initialised process group must hold the same schedule."""
    mine = schedule_digest(schedule)
    all_ = [None] * dist.get_world_size()
    dist.all_gather_object(all_, mine)
    if any(x != mine for x in all_):
        raise RuntimeError("ranks disagree on the arrival schedule")


def combine_gap_stats(sum_gap, max_gap, dist):
    """Gap statistics of a sharded master: every rank holds the sum and maximum of the Gap over
    its own range (ga_get_stats); the whole vector's are the sum of sums and the max of maxima.
    These two scalars per arrival are the only values ranks ever exchange, and only for logging."""
    import torch
    dev = "cuda" if dist.get_backend() == "nccl" else "cpu"
    s = torch.tensor([sum_gap], dtype=torch.float64, device=dev)
    m = torch.tensor([max_gap], dtype=torch.float64, device=dev)
    dist.all_reduce(s, op=dist.ReduceOp.SUM)
    dist.all_reduce(m, op=dist.ReduceOp.MAX)
    return float(s.item()), float(m.item())
