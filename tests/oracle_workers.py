"""Worker functions for the tests that fan the CPU oracle out over processes (started with spawn, so
that no worker is a fork of a process that has already talked to the GPU).  Each returns int8 rows:
schedule entries lie in [-31, 30], the batch form's padding is passed as -128."""
import os
import sys

import numpy as np

sys.path.insert(0, os.path.dirname(os.path.dirname(os.path.abspath(__file__))))


def recv_rows(job):
    """(p, root, lo, hi) -> receive rows of actual ranks [lo, hi) by Algorithm 5, int8."""
    import oracle
    p, root, lo, hi = job
    recv, _ = oracle.schedule_table(p, root, lo, hi, want_send=False)
    return recv.astype(np.int8)


def batch_rows(job):
    """(p[], rank[], root[]) -> (receive rows by Algorithm 5, send rows by Algorithm 6), int8, padded with -128."""
    import oracle
    p, rank, root = job
    recv, _ = oracle.schedule_batch(p, rank, root, 31, -128, want_send=False)
    send = oracle.sendschedule_alg6_batch(p, rank, root, 31, -128)
    return recv.astype(np.int8), send.astype(np.int8)


def pool_size() -> int:
    return max(1, min(os.cpu_count() or 1, 16))
