#!/usr/bin/env python
"""Writes tests/golden/checksums_2_65536.txt: the schedule checksum of every p in [2, 65536].

Calls nothing but the CPU oracle (oracle.checksum: both tables of p by Algorithm 5 and the
definition of the send schedule, then the wrapping sum of the SplitMix64-mixed (r, k, recv,
send) keys).  About 2.1e9 receive schedules: some 25 minutes of one core, a few minutes when
fanned out over the host's cores (one process per core, started with spawn).

    python tests/golden/make_checksums.py [processes]
"""
import multiprocessing as mp
import os
import sys
import time

HERE = os.path.dirname(os.path.abspath(__file__))
ROOT = os.path.dirname(os.path.dirname(HERE))
P_LO, P_HI = 2, 65536
OUT = os.path.join(HERE, "checksums_%d_%d.txt" % (P_LO, P_HI))


def work(block):
    sys.path.insert(0, ROOT)
    import oracle
    return [(p, oracle.checksum(p)) for p in block]


def main():
    procs = int(sys.argv[1]) if len(sys.argv) > 1 else (os.cpu_count() or 1)
    ps = list(range(P_HI, P_LO - 1, -1))                      # largest first: the long jobs start early
    blocks = [ps[i:i + 64] for i in range(0, len(ps), 64)]
    sys.path.insert(0, ROOT)
    import oracle
    oracle.build()
    t0 = time.time()
    sums = {}
    with mp.get_context("spawn").Pool(procs) as pool:
        for part in pool.imap_unordered(work, blocks):
            sums.update(part)
    with open(OUT, "w") as fh:
        fh.write("# checksum(p) of the broadcast schedule (root 0) for p = %d .. %d, one per line, hex;\n" % (P_LO, P_HI))
        fh.write("# written by tests/golden/make_checksums.py from the CPU oracle alone\n")
        for p in range(P_LO, P_HI + 1):
            fh.write("%016x\n" % sums[p])
    print("wrote %s in %.0f s with %d processes" % (OUT, time.time() - t0, procs))


if __name__ == "__main__":
    main()
