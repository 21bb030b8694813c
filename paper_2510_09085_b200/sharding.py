"""Partition of a batch of utterances over GPUs.

Algorithm 1 decodes one utterance at a time and nothing is shared between
utterances, so a batch shards over devices by its batch dimension with no
exchange step: every rank decodes its own utterances with the single-GPU
library and the results are concatenated (or simply kept where they are).

A rank is busy for as long as its longest frame chain and its total number of
frames keep it, so the split balances total frames: longest utterance first,
each to the shard that holds the fewest frames so far (the classical
longest-processing-time-first rule).  The rule is deterministic, so every rank
computes the same partition from the lengths alone and no rank has to be told
its share.
"""
from __future__ import annotations

import heapq

import numpy as np


def lpt_shards(lengths, n_shards: int) -> list[np.ndarray]:
    """Indices of the utterances of each of ``n_shards`` shards (each sorted ascending).

    Longest first, each to the currently lightest shard; ties go to the lower shard and, among
    utterances of equal length, to the lower index, so the result depends on ``lengths`` only.
    Every utterance lands in exactly one shard.  The heaviest and the lightest shard differ by
    at most the longest utterance in total frames (and any shard holds at most
    ``total / n_shards + longest`` frames)."""
    lengths = np.asarray(lengths, dtype=np.int64)
    if n_shards < 1:
        raise ValueError("n_shards must be at least 1")
    order = sorted(range(len(lengths)), key=lambda i: (-int(lengths[i]), i))
    heap = [(0, s) for s in range(n_shards)]          # (frames so far, shard)
    heapq.heapify(heap)
    members: list[list[int]] = [[] for _ in range(n_shards)]
    for i in order:
        load, s = heapq.heappop(heap)
        members[s].append(i)
        heapq.heappush(heap, (load + max(0, int(lengths[i])), s))
    return [np.array(sorted(m), dtype=np.int64) for m in members]


def shard_of_rank(lengths, rank: int, world: int) -> np.ndarray:
    """The utterances rank ``rank`` of ``world`` decodes."""
    return lpt_shards(lengths, world)[rank]
