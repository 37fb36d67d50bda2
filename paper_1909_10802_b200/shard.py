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


def layer_shard_range(layer_offsets, rank, world):
    """(l0, l1, j0, n): rank `rank` owns the whole layers l0 .. l1-1, i.e. parameters [j0, j0+n).

    The layer-wise Gap (Section 5.3) needs the norm of a whole layer, and the layers are independent
    of one another, so ranks that hold whole layers need no exchange either. layer_offsets are the
    len(layers)+1 ascending offsets of the layers in the vector. The cut before rank r is the layer
    boundary nearest to r/world of the vector, moved where needed so that every rank owns at least
    one layer; the ranges tile the vector exactly. A vector dominated by one layer cannot be balanced
    this way (that layer stays on one rank)."""
    off = [int(x) for x in layer_offsets]
    n_layers = len(off) - 1
    if n_layers < 1 or any(b <= a for a, b in zip(off, off[1:])) or off[0] != 0:
        raise ValueError("layer_offsets must ascend from 0 and name at least one non-empty layer")
    if not (0 <= rank < world):
        raise ValueError("rank out of range")
    if world > n_layers:
        raise ValueError("more ranks than layers: a layer is not split")
    d = off[-1]
    cuts = [0]
    for r in range(1, world):
        ideal = d * r / world
        lo, hi = cuts[-1] + 1, n_layers - (world - r)        # leave one layer for everyone before and after
        best = min(range(lo, hi + 1), key=lambda l: (abs(off[l] - ideal), l))
        cuts.append(best)
    cuts.append(n_layers)
    l0, l1 = cuts[rank], cuts[rank + 1]
    return l0, l1, off[l0], off[l1] - off[l0]


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
