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
