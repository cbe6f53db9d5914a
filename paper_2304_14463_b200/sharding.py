"""Host-side helpers for running one batch on several GPUs: sequences are independent, so a batch
is cut into contiguous blocks, one per rank, the (small) graph is replicated, and no collective is
needed to evaluate; gathering the 20 bytes of output per sequence is optional."""
from __future__ import annotations

import numpy as np


def shard_range(B: int, rank: int, world: int):
    """Half-open range [b0, b1) of the sequences rank ``rank`` of ``world`` evaluates."""
    if not (0 <= rank < world):
        raise ValueError("rank outside [0, world)")
    return B * rank // world, B * (rank + 1) // world


def shard_batch(seqs: np.ndarray, lens: np.ndarray, rank: int, world: int):
    """Packed (seqs, lens) of the block of rank ``rank``; views, no copy of the sequence data."""
    b0, b1 = shard_range(len(lens), rank, world)
    clipped = np.clip(lens, 0, None).astype(np.int64)
    offs = np.concatenate([[0], np.cumsum(clipped)])
    return seqs[offs[b0]:offs[b1]], lens[b0:b1]


def aggregate_throughput(units_per_rank, seconds_per_rank):
    """Whole-job throughput: all units processed divided by the slowest rank's time."""
    return float(np.sum(units_per_rank)) / float(np.max(seconds_per_rank))


def best_over_ranks(best: dict, M: int, first_chain: int, max_len: int, device="cpu", group=None):
    """Best chain of a population split over the ranks of a process group (the chains themselves
    never leave their rank).

    ``best`` is this rank's best chain as a dict with ``index`` (local, -1 when the rank has no
    valid chain), ``peak``, ``dur``, ``status`` and ``seq`` (1-D int array); ``first_chain`` the
    global number of the rank's chain 0.  Every rank gets the same answer: the chain with the
    smallest key (max(peak, M), dur), lowest global number among equals, as a dict with the global
    ``index``, ``rank`` (owner), ``peak``, ``dur``, ``status`` and ``seq``; ``index`` = -1 when no
    rank has a valid chain.  Cost: one all-gather of six integers per rank and one broadcast of
    max_len integers."""
    import torch
    import torch.distributed as dist
    world = dist.get_world_size(group)
    valid = best["index"] >= 0
    big = (1 << 62)
    mine = torch.tensor([max(int(best["peak"]), int(M)) if valid else big, int(best["dur"]) if valid else big,
                         first_chain + int(best["index"]) if valid else big, int(best["peak"]), int(best["status"]),
                         len(best["seq"]) if valid else 0], dtype=torch.int64, device=device)
    allv = [torch.empty_like(mine) for _ in range(world)]
    dist.all_gather(allv, mine, group=group)
    rows = [tuple(int(x) for x in v.tolist()) for v in allv]
    owner = min(range(world), key=lambda r: rows[r][:3])
    a, d, gidx, peak, status, length = rows[owner]
    if gidx == big:
        return dict(index=-1, rank=-1, peak=-1, dur=-1, status=-2, seq=np.zeros(0, np.int32))
    buf = torch.zeros(max_len, dtype=torch.int32, device=device)
    if dist.get_rank(group) == owner:
        buf[:length] = torch.as_tensor(np.asarray(best["seq"], np.int32), device=device)
    src = owner if group is None else dist.get_global_rank(group, owner)
    dist.broadcast(buf, src=src, group=group)
    return dict(index=gidx, rank=owner, peak=peak, dur=d, status=status, seq=buf[:length].cpu().numpy())
