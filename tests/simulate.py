"""Brute-force round-by-round simulation of the n-block broadcast (Algorithm 1).

Test-side checker: it moves blocks between p simulated processors exactly as
the schedule tables dictate and records what each processor holds.  The rules
the paper leaves to the Send||Recv operation are applied here: a negative block
is neither sent nor received, a block above n-1 stands for block n-1, nothing
is sent to the root, and the root receives nothing.
"""
from __future__ import annotations

import numpy as np


def simulate(p, n, root, skip, recv_tab, send_tab, rounds_of):
    """Run the broadcast.

    recv_tab/send_tab: [p][q] tables indexed by ACTUAL rank.
    rounds_of(recv_row, send_row) -> (k[], raw_recv[], raw_send[]) per communication round.
    Returns a dict of facts; raises AssertionError on any inconsistency.
    """
    q = recv_tab.shape[1]
    total = n - 1 + q
    held = np.zeros((p, n), dtype=bool)
    held[root, :] = True
    times_received = np.zeros((p, n), dtype=np.int64)
    per_rank = [rounds_of(recv_tab[a], send_tab[a]) for a in range(p)]
    done_round = None
    for j in range(total):
        # what every processor puts on the wire this round, from its state BEFORE the round
        outgoing = {}
        for a in range(p):
            k = int(per_rank[a][0][j])
            raw = int(per_rank[a][2][j])
            to = (a + int(skip[k])) % p
            if raw < 0 or to == root:
                continue
            blk = min(raw, n - 1)
            assert held[a, blk], f"p={p} n={n} round {j}: rank {a} sends block {blk} it does not hold"
            outgoing[(a, to)] = blk
        arrivals = []
        for a in range(p):
            k = int(per_rank[a][0][j])
            raw = int(per_rank[a][1][j])
            frm = (a - int(skip[k])) % p
            if a == root or raw < 0:
                # whatever the from-processor sends would be lost: it must not send a real block
                assert (frm, a) not in outgoing or a != root, "block sent to root"
                if a != root:
                    assert (frm, a) not in outgoing, (
                        f"p={p} n={n} round {j}: rank {frm} sends to {a}, which expects nothing")
                continue
            blk = min(raw, n - 1)
            assert outgoing.get((frm, a)) == blk, (
                f"p={p} n={n} round {j}: rank {a} expects block {blk} from {frm}, "
                f"which sends {outgoing.get((frm, a))}")
            arrivals.append((a, blk))
        for a, blk in arrivals:
            times_received[a, blk] += 1
            held[a, blk] = True
        if done_round is None and held.all():
            done_round = j + 1
    return dict(done_round=done_round, held=held, times_received=times_received, total=total)
