"""Seeded synthetic workloads: process counts and query batches.

Only input generation lives here -- nothing of the schedule arithmetic -- so
that the CUDA path and the CPU checker can be fed the very same arrays.
"""
from __future__ import annotations

import numpy as np

# Process counts shaped like the paper's experiments (200 .. 25 600 MPI processes,
# schedule timings up to ~2.1 M and ~16 M processors), extended to 2^27.
P_SMALL = 1000                     # q = 10
P_MEDIUM = 2 ** 20 + 1             # q = 21, almost every rank has Algorithm 6 violations
P_LARGE = 2 ** 27 - 1              # q = 27, ~29 GB of tables
SWEEP_RANGE = (2, 65536)           # exhaustive verification sweep
N_QUERIES = 2 ** 24                # random query batch


def query_batch(nq: int = N_QUERIES, seed: int = 0):
    """(p, rank, root) int32 arrays: p log-uniform in [2, 2^31-1], rank and root uniform in [0, p)."""
    rng = np.random.default_rng(seed)
    p = np.floor(np.exp2(rng.uniform(1.0, 31.0, nq))).astype(np.int64)
    p = np.clip(p, 2, 2 ** 31 - 1)
    rank = np.minimum(np.floor(rng.random(nq) * p).astype(np.int64), p - 1)
    root = np.minimum(np.floor(rng.random(nq) * p).astype(np.int64), p - 1)
    return p.astype(np.int32), rank.astype(np.int32), root.astype(np.int32)


def sample_ranks(p: int, count: int, seed: int = 0) -> np.ndarray:
    """Sorted sample of ranks of [0, p): both ends, powers of two and their neighbours, random fill."""
    rng = np.random.default_rng(seed)
    fixed = [0, 1, 2, p - 1, p - 2, p // 2]
    k = 1
    while k < p:
        fixed += [k - 1, k, k + 1]
        k *= 2
    fixed = [r for r in fixed if 0 <= r < p]
    rnd = rng.integers(0, p, max(count - len(fixed), 0)).tolist()
    return np.unique(np.array(fixed + rnd, dtype=np.int64))


def sample_windows(p: int, width: int, count: int, seed: int = 0):
    """Start ranks of `count` windows of `width` consecutive ranks, multiples of 32, plus both ends."""
    rng = np.random.default_rng(seed)
    last = max(p - width, 0)
    starts = [0, last // 32 * 32] + (rng.integers(0, last // 32 + 1, count) * 32).tolist()
    return sorted(set(int(s) for s in starts))
