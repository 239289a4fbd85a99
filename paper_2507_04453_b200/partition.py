"""Candidate sharding for multi-GPU runs (host logic only).

Candidates are independent (Algorithm 1, line 4: workers run "in parallel"; every worker holds the same
frozen weights and CMA-ES state), so a population is split into contiguous candidate ranges, one per rank,
balanced by token count.  Each rank regenerates the singular values of its own candidates from <seed, k>
(essa_sample_population_range) and projects its own tokens; there is no collective on the data path.
The only exchange in the surrounding loop is Algorithm 1, line 11: <seed, reward> pairs, 8 bytes per candidate.
"""
from __future__ import annotations

from typing import List, Tuple

import numpy as np


def partition_candidates(seg_offsets, world_size: int) -> List[Tuple[int, int]]:
    """Contiguous candidate ranges [k_begin, k_end) per rank, balanced by tokens.

    Rank g gets the candidates whose token midpoint falls in the g-th equal slice of the token axis;
    every candidate lands on exactly one rank and ranges are ordered.  With no tokens at all the split
    is by candidate count.
    """
    off = np.asarray(seg_offsets, dtype=np.int64)
    P = off.shape[0] - 1
    T = int(off[-1]) if P >= 0 else 0
    if world_size <= 0:
        raise ValueError("world_size must be positive")
    if T == 0:
        cuts = [(P * g) // world_size for g in range(world_size + 1)]
    else:
        mid2 = off[:-1] + off[1:]  # twice the midpoint, exact integers
        cuts = [0]
        for g in range(1, world_size):
            cuts.append(int(np.searchsorted(mid2, 2 * T * g / world_size, side="left")))
        cuts.append(P)
        for g in range(1, world_size + 1):  # keep ranges ordered
            cuts[g] = max(cuts[g], cuts[g - 1])
    return [(cuts[g], cuts[g + 1]) for g in range(world_size)]


def local_offsets(seg_offsets, k_begin: int, k_end: int) -> np.ndarray:
    """Segment offsets of a rank's own candidates, rebased so that its first token is 0."""
    off = np.asarray(seg_offsets, dtype=np.int64)
    return (off[k_begin:k_end + 1] - off[k_begin]).astype(np.int32)


def pack_seed_reward(seed: int, reward: float) -> np.ndarray:
    """One <seed, reward> message: a 32-bit seed and a 32-bit float reward (8 bytes)."""
    out = np.zeros(2, dtype=np.uint32)
    out[0] = np.uint32(seed & 0xFFFFFFFF)
    out[1] = np.array([reward], dtype=np.float32).view(np.uint32)[0]
    return out
