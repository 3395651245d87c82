"""Pins for the CPU oracle: everything the paper and the mathematics fix about
the schedule, checked without reference to the CUDA path."""
import numpy as np
import pytest

import oracle
from conftest import load_golden
from simulate import simulate

RNG = np.random.default_rng(12345)
BIG_P = [2 ** 20 + 1, 2 ** 20, 2 ** 20 - 1, 2 ** 27 - 1, 2 ** 24 + 3, 2 ** 31 - 1, 2 ** 30 + 1,
         1000003, 16 * 2 ** 20 + 12345]


def ctz(x):
    return (x & -x).bit_length() - 1


# ---------------------------------------------------------------- printed tables
@pytest.mark.parametrize("name", ["table1_p17.txt", "table2_p9.txt", "table3_p18.txt"])
def test_printed_tables(name):
    d = load_golden(name)
    p, q = d["p"][0], d["q"][0]
    assert oracle.q_of(p) == q
    recv, send = oracle.schedule_table(p)
    for k in range(q):
        assert recv[:, k].tolist() == d[f"recv{k}"], f"recvblock[{k}]"
        assert send[:, k].tolist() == d[f"send{k}"], f"sendblock[{k}]"
    assert [oracle.baseblock(p, r) for r in range(p)] == d["b"]
    for r in range(p):
        assert oracle.recvschedule(p, r).tolist() == [d[f"recv{k}"][r] for k in range(q)]
        assert oracle.sendschedule(p, r).tolist() == [d[f"send{k}"][r] for k in range(q)]
        assert oracle.sendschedule_alg6(p, r)[0].tolist() == [d[f"send{k}"][r] for k in range(q)]


def test_printed_baseblock_listing_p11():
    d = load_golden("baseblocks_p11.txt")
    assert oracle.skips(11).tolist() == d["skips"]
    assert [oracle.baseblock(11, r) for r in range(11)] == d["b"]


def test_printed_skips_p17():
    d = load_golden("skips_p17.txt")
    assert oracle.skips(17).tolist() == d["skips"]


# ---------------------------------------------------------------- skips (Algorithm 2)
def test_skip_facts():
    ps = list(range(2, 3000)) + [int(x) for x in RNG.integers(3000, 2 ** 31 - 1, 3000)] + BIG_P
    for p in ps:
        s = oracle.skips(p).tolist()
        q = len(s) - 1
        assert 2 ** (q - 1) < p <= 2 ** q
        assert s[0] == 1 and s[1] == 2 and s[q] == p          # stated after Algorithm 2
        for k in range(q):
            assert s[k + 1] <= 2 * s[k] <= s[k + 1] + 1           # Observation 3
            assert s[k] == -(-s[k + 1] // 2)                      # ceil-halving
            tot = sum(s[: k + 1])
            assert s[k + 1] - 1 <= tot < s[k + 1] + k             # Lemma 1
            assert s[k] == -(-p // 2 ** (q - k))                  # halving composes
    assert oracle.skips(1).tolist() == [1]
    assert oracle.q_of(1) == 0 and oracle.q_of(2) == 1 and oracle.q_of(3) == 2
    assert oracle.q_of(2 ** 31 - 1) == 31 and oracle.q_of(2 ** 27 - 1) == 27
    assert oracle.q_of(2 ** 20 + 1) == 21


# ---------------------------------------------------------------- baseblock (Algorithm 3)
def test_baseblock_power_of_two_is_ctz():
    for q in range(1, 12):
        p = 2 ** q
        assert oracle.baseblock(p, 0) == q
        for r in range(1, p):
            assert oracle.baseblock(p, r) == ctz(r)


def test_baseblock_listing_by_self_append():
    """Proof of Lemma 3: the list for skip[k+1] processors is the list for skip[k]
    appended to itself, possibly minus its last element, with entry 0 raised to k+1."""
    for p in list(range(2, 600)) + [1000, 4097, 65537]:
        s = oracle.skips(p).tolist()
        q = len(s) - 1
        lst = [0]
        for k in range(q):
            lst = (lst + lst)[: s[k + 1]]
            lst[0] = k + 1
        assert len(lst) == p
        assert lst == [oracle.baseblock(p, r) for r in range(p)]


def test_baseblock_is_first_index_of_a_skip_sequence():
    """b_r < q for r>0, and r - skip[b_r] is reachable with larger indices only."""
    for p in [5, 17, 100, 1000, 4099]:
        s = oracle.skips(p).tolist()
        q = len(s) - 1
        for r in range(1, p):
            b = oracle.baseblock(p, r)
            assert 0 <= b < q
            # greedy remainder uses only indices > b
            rem, k = r, q
            used = []
            while rem and k > 0:
                k -= 1
                rp = r - rem
                if rp + s[k] <= r:
                    rem -= s[k]
                    used.append(k)
            assert rem == 0 and min(used) == b


def test_lemma3_windows():
    """Lemma 3's proof: the first skip[k] baseblocks hold exactly k+1 different values.
    (The lemma's printed bound for ANY window of that length is too strong by one:
    p=9 has baseblocks 0,3,0 at r=4..6, a window of skip[2]=3 with two values; what
    holds for every window is at least k.)"""
    assert [oracle.baseblock(9, r) for r in (4, 5, 6)] == [0, 3, 0]
    for p in [9, 17, 18, 33, 100, 257, 1000]:
        s = oracle.skips(p).tolist()
        q = len(s) - 1
        b = [oracle.baseblock(p, r) for r in range(p)]
        for k in range(q):
            w = s[k]
            assert len(set(b[0:w])) == k + 1
            for r in range(0, p - w + 1):
                assert len(set(b[r:r + w])) >= k


# ---------------------------------------------------------------- the four conditions
def check_conditions(p, recv, send):
    s = oracle.skips(p)
    q = len(s) - 1
    ranks = np.arange(p)
    b = np.array([oracle.baseblock(p, r) for r in range(p)]) if p <= 5000 else None
    for k in range(q):
        f = (ranks - s[k]) % p
        t = (ranks + s[k]) % p
        assert np.array_equal(recv[:, k], send[f, k]), "condition 1"
        assert np.array_equal(send[:, k], recv[t, k]), "condition 2"
    # condition 3: set equality; the root has no non-negative entry
    srt = np.sort(recv, axis=1)
    assert np.array_equal(srt[0], np.arange(-q, 0)), "root receives {-q..-1}"
    nonneg = (recv >= 0).sum(axis=1)
    assert nonneg[0] == 0 and (nonneg[1:] == 1).all()
    base = recv.max(axis=1)
    if b is not None:
        assert np.array_equal(base[1:], b[1:])
    for r in range(1, min(p, 3000)):
        want = sorted((set(range(-q, 0)) - {int(base[r]) - q}) | {int(base[r])})
        assert srt[r].tolist() == want, "condition 3"
    # condition 4 and its corollary
    assert np.array_equal(send[0], np.arange(q)), "root sends block k in round k"
    assert np.array_equal(send[1:, 0], base[1:] - q), "sendblock[0] = b - q"
    for k in range(1, q):
        ok = send[1:, k] == (base[1:] - q)
        for j in range(k):
            ok |= send[1:, k] == recv[1:, j]
        assert ok.all(), "condition 4"


def test_conditions_small_p_exhaustive():
    for p in range(2, 400):
        recv, send = oracle.schedule_table(p)
        check_conditions(p, recv, send)


@pytest.mark.parametrize("p", [1000, 4097, 8191, 12345, 65537])
def test_conditions_larger_p(p):
    recv, send = oracle.schedule_table(p)
    check_conditions(p, recv, send)


# ---------------------------------------------------------------- closed form for p = 2^q
def test_power_of_two_closed_form():
    """For p = 2^q the doubling observations give, by induction from p = 2:
    send[k]_r = b_r if r < 2^k (k for the root), else ctz(r with its low k bits cleared) - q;
    recv[k]_r = send[k] of (r - 2^k) mod p."""
    for q in range(1, 12):
        p = 2 ** q
        recv, send = oracle.schedule_table(p)
        for r in range(p):
            for k in range(q):
                if r < 2 ** k:
                    want = k if r == 0 else ctz(r)
                else:
                    want = ctz(r & ~(2 ** k - 1)) - q
                assert send[r, k] == want
                f = (r - 2 ** k) % p
                if f < 2 ** k:
                    wr = k if f == 0 else ctz(f)
                else:
                    wr = ctz(f & ~(2 ** k - 1)) - q
                assert recv[r, k] == wr


# ---------------------------------------------------------------- doubling (Observations 2 and 6)
def test_doubling_receive_schedule():
    for p in range(2, 300):
        q = oracle.q_of(p)
        recv, _ = oracle.schedule_table(p)
        recv2, _ = oracle.schedule_table(2 * p)
        assert oracle.q_of(2 * p) == q + 1
        built = np.zeros((2 * p, q + 1), dtype=np.int64)
        built[:p, :q] = recv
        built[p:, :q] = recv
        built[:, :q] -= (built[:, :q] < 0)
        built[:p, q] = -1
        built[p, q] = q
        # r = p copies the root's row, which has no non-negative entry
        for r in range(p + 1, 2 * p):
            row = built[r, :q]
            k = int(np.argmax(row >= 0))
            assert row[k] >= 0
            built[r, q] = row[k]
            row[k] = -1
        assert np.array_equal(built, recv2), f"Observation 2 fails for p={p}"


def test_doubling_send_schedule():
    for p in range(2, 300):
        q = oracle.q_of(p)
        _, send = oracle.schedule_table(p)
        _, send2 = oracle.schedule_table(2 * p)
        b = [oracle.baseblock(p, r) for r in range(p)]
        built = np.zeros((2 * p, q + 1), dtype=np.int64)
        built[:p, :q] = send
        built[p:, :q] = send
        built[:, :q] -= (built[:, :q] < 0)
        built[:p, q] = b
        built[0, q] = q           # the root keeps sending block k in round k
        hi = built[p:, :q]
        hi[hi >= 0] = -1
        built[p:, q] = -1
        assert np.array_equal(built, send2), f"Observation 6 fails for p={p}"


# ---------------------------------------------------------------- Algorithm 6 against the definition
def test_alg6_equals_definition_small():
    for p in range(1, 500):
        _, send = oracle.schedule_table(p)
        for r in range(p):
            row, viol, _ = oracle.sendschedule_alg6(p, r)
            assert row.tolist() == send[r].tolist(), (p, r)
            assert viol <= 4                                        # Theorem 3


def test_alg6_equals_definition_large_sampled():
    for p in BIG_P:
        for r in [0, 1, 2, p - 1, p - 2, p // 2] + [int(x) for x in RNG.integers(0, p, 150)]:
            row, viol, _ = oracle.sendschedule_alg6(p, r)
            assert row.tolist() == oracle.sendschedule(p, r).tolist(), (p, r)
            assert viol <= 4


def test_stated_violation_p17():
    # Section 2.3 names a violation in round 2 for processor 3 of p=17.
    _, viol, mask = oracle.sendschedule_alg6(17, 3)
    assert viol >= 1 and mask & (1 << 2)


# ---------------------------------------------------------------- bounds (Lemmas 5, 6)
def test_search_bounds():
    ps = list(range(2, 700)) + BIG_P
    for p in ps:
        q = oracle.q_of(p)
        ranks = range(p) if p < 700 else [0, 1, p - 1] + [int(x) for x in RNG.integers(0, p, 200)]
        for r in ranks:
            row, st = oracle.recvschedule(p, r, with_stats=True)
            assert st["oob"] == 0
            assert st["calls"] <= max(q - 1, 0)                     # Lemma 5
            assert st["retest_hits"] == 0                           # the repeated test never passes
            assert st["iters"] - st["retests"] <= 2 * q + st["calls"]   # Lemma 6
            assert (row > -1000 + 64).all()                         # every entry was written


def test_lemma4_intermediate_processors():
    """Lemma 4: r - skip[k+1] <= r'_k <= r - skip[k] (on p + r), strictly decreasing in k, and
    recvblock[k] is the baseblock of r'_k (the root's own index q standing for b)."""
    ps = list(range(2, 300)) + BIG_P
    for p in ps:
        s = oracle.skips(p).tolist()
        q = len(s) - 1
        ranks = range(p) if p < 300 else [0, 1, p - 1] + [int(x) for x in RNG.integers(0, p, 100)]
        for r in ranks:
            pos = oracle.recv_positions(p, r).tolist()
            row = oracle.recvschedule(p, r).tolist()
            b = oracle.baseblock(p, r)
            for k in range(q):
                assert p + r - s[k + 1] <= pos[k] <= p + r - s[k], (p, r, k)
                if k > 0:
                    assert pos[k] < pos[k - 1]
                # the accepted index is the first index of the path to r'_k, which starts with skip[q] = p
                if pos[k] == p:
                    assert row[k] == b
                elif p < 300:
                    assert row[k] + q >= 0 and row[k] < 0


# ---------------------------------------------------------------- table modes and root renumbering
def test_table_modes_agree_and_root():
    for p, root in [(17, 0), (17, 5), (100, 99), (1000, 123), (1025, 7)]:
        recv0, send0 = oracle.schedule_table(p, 0)
        recv, send = oracle.schedule_table(p, root)
        idx = (np.arange(p) - root) % p
        assert np.array_equal(recv, recv0[idx]) and np.array_equal(send, send0[idx])
        lo, hi = p // 3, p // 3 + 40
        recv_w, send_w = oracle.schedule_table(p, root, lo, min(hi, p))
        assert np.array_equal(recv_w, recv[lo:hi]) and np.array_equal(send_w, send[lo:hi])
        _, send_only = oracle.schedule_table(p, root, want_recv=False)
        assert np.array_equal(send_only, send)
        for a in range(0, p, max(1, p // 17)):
            r = (a - root) % p
            assert oracle.recvschedule(p, r).tolist() == recv[a].tolist()
            assert oracle.sendschedule(p, r).tolist() == send[a].tolist()


def test_degenerate_p():
    recv, send = oracle.schedule_table(1)
    assert recv.shape == (1, 0) and send.shape == (1, 0)
    recv, send = oracle.schedule_table(2)
    assert recv.tolist() == [[-1], [0]] and send.tolist() == [[0], [-1]]
    with pytest.raises(ValueError):
        oracle.schedule_table(0)
    with pytest.raises(ValueError):
        oracle.schedule_table(5, 5)
    with pytest.raises(ValueError):
        oracle.schedule_table(5, 0, 3, 6)


# ---------------------------------------------------------------- Algorithm 1: lookup and simulation
def test_round_lookup_matches_printed_loop():
    for q in range(1, 9):
        for n in range(1, 30):
            row = RNG.integers(-q, q, q).astype(np.int32)
            x, k, rr, sr = oracle.broadcast_rounds(q, n, row, row)
            assert x == (q - (n - 1) % q) % q
            assert (x + n - 1 + q) % q == 0                         # last round ends a phase
            for j in range(n - 1 + q):
                i = x + j
                assert k[j] == i % q == oracle.round_k(q, n, j)
                assert rr[j] == row[i % q] + q * (i // q) - x        # Theorem 1
                want = -1 if rr[j] < 0 else min(int(rr[j]), n - 1)
                assert oracle.round_block(q, n, j, row) == want
            assert oracle.round_block(q, n, n - 1 + q, row) == -2
            assert oracle.round_block(q, n, -1, row) == -2


def _run_sim(p, n, root):
    recv, send = oracle.schedule_table(p, root)
    q = recv.shape[1]
    skip = oracle.skips(p)

    def rounds_of(rrow, srow):
        _, k, rr, sr = oracle.broadcast_rounds(q, n, rrow, srow)
        return k, rr, sr

    res = simulate(p, n, root, skip, recv, send, rounds_of)
    assert res["held"].all(), f"p={p} n={n}: some block missing after {res['total']} rounds"
    assert res["done_round"] == n - 1 + q, f"p={p} n={n}: finished in {res['done_round']} rounds"
    tr = res["times_received"]
    assert (tr[root] == 0).all()
    others = np.delete(tr, root, axis=0)
    assert (others == 1).all(), f"p={p} n={n}: a block was received {others.max()} times"


def test_simulation_tiny_exhaustive():
    for p in range(2, 65):
        for n in range(1, 11):
            _run_sim(p, n, 0)


def test_simulation_other_roots_and_p1000():
    _run_sim(17, 8, 5)
    _run_sim(33, 13, 32)
    _run_sim(1000, 8, 0)          # 8 blocks over 17 rounds


# ---------------------------------------------------------------- checksum and batch forms
def _mix(z):
    z = np.uint64(z)
    z ^= z >> np.uint64(30)
    z *= np.uint64(0xBF58476D1CE4E5B9)
    z ^= z >> np.uint64(27)
    z *= np.uint64(0x94D049BB133111EB)
    z ^= z >> np.uint64(31)
    return z


def test_checksum_definition():
    with np.errstate(over="ignore"):
        for p in [2, 3, 17, 100, 1000]:
            recv, send = oracle.schedule_table(p)
            q = recv.shape[1]
            r = np.arange(p, dtype=np.uint64)[:, None]
            k = np.arange(q, dtype=np.uint64)[None, :]
            key = (r << np.uint64(32)) | (k << np.uint64(16)) \
                | ((recv.astype(np.int64) & 0xFF).astype(np.uint64) << np.uint64(8)) \
                | (send.astype(np.int64) & 0xFF).astype(np.uint64)
            want = int(_mix(key).sum(dtype=np.uint64))
            assert oracle.checksum(p) == want
    # SplitMix64 finaliser applied to the first state 0x9e3779b97f4a7c15 gives the
    # generator's published first output for seed 0.
    with np.errstate(over="ignore"):
        assert int(_mix(np.uint64(0x9E3779B97F4A7C15))) == 0xE220A8397B1DCDAF
    assert oracle.checksum(1) == 0


def test_batch_form():
    p = np.array([2, 17, 1000, 2 ** 20 + 1, 2 ** 31 - 1, 1], dtype=np.int32)
    rank = np.array([1, 3, 999, 12345, 2 ** 31 - 2, 0], dtype=np.int32)
    root = np.array([0, 5, 500, 2 ** 20, 17, 0], dtype=np.int32)
    recv, send = oracle.schedule_batch(p, rank, root)
    assert recv.shape == (6, 31)
    for i in range(6):
        q = oracle.q_of(int(p[i]))
        r = (int(rank[i]) - int(root[i])) % int(p[i])
        assert recv[i, :q].tolist() == oracle.recvschedule(int(p[i]), r).tolist()
        assert send[i, :q].tolist() == oracle.sendschedule_alg6(int(p[i]), r)[0].tolist()
        assert (recv[i, q:] == oracle.PAD).all() and (send[i, q:] == oracle.PAD).all()


# ---------------------------------------------------------------- Algorithm 7: all-broadcast tables
def test_allbroadcast_tables_are_renumbered_broadcast_tables():
    """Processor r with root j is virtual rank (r - j) mod p of the broadcast from root j."""
    for p in [2, 3, 9, 17, 18, 100, 257]:
        per_root = [oracle.schedule_table(p, root) for root in range(p)]
        for r in sorted({0, 1, p // 2, p - 1}):
            recv, send = oracle.allbroadcast_schedule(p, r)
            for j in range(p):
                assert recv[j].tolist() == per_root[j][0][r].tolist()
                assert send[j].tolist() == per_root[j][1][r].tolist()
            lo, hi = p // 3, min(p, p // 3 + 7)
            recv_w, send_w = oracle.allbroadcast_schedule(p, r, lo, hi)
            assert np.array_equal(recv_w, recv[lo:hi]) and np.array_equal(send_w, send[lo:hi])


def test_allbroadcast_simulation():
    """Algorithm 7 round by round on tiny systems: every processor ends with all n blocks of every
    other processor after n-1+q rounds, what it unpacks for root j is what its from-processor packed
    for root j, and nobody packs a block it does not hold."""
    for p in list(range(2, 14)) + [17, 18]:
        q = oracle.q_of(p)
        skip = oracle.skips(p)
        tables = [oracle.allbroadcast_schedule(p, r) for r in range(p)]
        for n in (1, 2, 3, 5, 8):
            x = (q - (n - 1) % q) % q
            held = np.zeros((p, p, n), dtype=bool)          # held[r][j][b]: r has block b of root j
            for r in range(p):
                held[r, r, :] = True
            # Algorithm 7's shift of all entries by -x, +q for the rounds before x
            sched = []
            for r in range(p):
                recv = tables[r][0].astype(np.int64) - x
                send = tables[r][1].astype(np.int64) - x
                recv[:, :x] += q
                send[:, :x] += q
                sched.append((recv, send))
            for i in range(x, n + q - 1 + x):
                k = i % q
                packed = {}
                for r in range(p):
                    t = (r + int(skip[k])) % p
                    for j in range(p):
                        if j != t:
                            raw = int(sched[r][1][j, k])
                            if raw >= 0:
                                blk = min(raw, n - 1)
                                assert held[r, j, blk], (p, n, i, r, j, blk)
                                packed[(r, j)] = blk
                        sched[r][1][j, k] += q
                arrivals = []
                for r in range(p):
                    f = (r - int(skip[k])) % p
                    for j in range(p):
                        if j != r:
                            raw = int(sched[r][0][j, k])
                            if raw >= 0:
                                blk = min(raw, n - 1)
                                assert packed.get((f, j)) == blk, (p, n, i, r, j, blk, packed.get((f, j)))
                                arrivals.append((r, j, blk))
                            else:
                                assert (f, j) not in packed or j == r, (p, n, i, r, j)
                        sched[r][0][j, k] += q
                for r, j, blk in arrivals:
                    held[r, j, blk] = True
            assert held.all(), (p, n)


# ---------------------------------------------------------------- Algorithm 1 by all processors; its reversal
def _arrival_by_theorem1(p, n, root, recv):
    """Theorem 1 read backwards: processor a receives block recv[k] + q*floor(i/q) - x in round i = x + j
    whatever the others do, so the round each block arrives in follows from a's own row."""
    q = recv.shape[1]
    arrival = np.full((n, p), -1, dtype=np.int64)
    arrival[:, root] = 0
    if q == 0:
        return arrival
    x = (q - (n - 1) % q) % q
    for a in range(p):
        if a == root:
            continue
        for j in range(n - 1 + q):
            i = x + j
            raw = int(recv[a, i % q]) + q * (i // q) - x
            if raw >= 0:
                blk = min(raw, n - 1)
                assert arrival[blk, a] == -1, "a block would arrive twice"
                arrival[blk, a] = j + 1
    return arrival


def test_simulated_broadcast_of_correct_tables():
    for p in list(range(1, 41)) + [63, 64, 65, 100]:
        q = oracle.q_of(p)
        for n in [1, 2, 3, q, q + 1, 2 * q + 3, 11]:
            if n < 1:
                continue
            for root in {0, p // 3, p - 1}:
                recv, send = oracle.schedule_table(p, root)
                arrival, stats = oracle.simulate_broadcast(p, root, n, recv, send)
                assert list(stats[:6]) == [0] * 6, (p, n, root, stats)
                assert stats[6] == (p - 1) * n
                assert stats[7] == (n - 1 + q if p > 1 else 0)        # the optimal number of rounds, all used
                assert (arrival == _arrival_by_theorem1(p, n, root, recv)).all()
                assert arrival.max() <= n - 1 + q and (arrival[:, root] == 0).all()


def test_simulated_broadcast_power_of_two_single_block():
    # one block on p = 2^q processors: processor r is reached in round floor(log2 r) + 1
    for q in range(1, 9):
        p = 1 << q
        recv, send = oracle.schedule_table(p)
        arrival, stats = oracle.simulate_broadcast(p, 0, 1, recv, send)
        assert list(arrival[0]) == [0] + [r.bit_length() for r in range(1, p)]
        assert stats[7] == q


def test_simulated_broadcast_agrees_with_the_brute_force_checker():
    for p, n, root in [(17, 8, 5), (33, 13, 32), (57, 6, 0), (1000, 8, 0)]:
        recv, send = oracle.schedule_table(p, root)
        q = recv.shape[1]

        def rounds_of(rrow, srow):
            _, k, rr, sr = oracle.broadcast_rounds(q, n, rrow, srow)
            return k, rr, sr

        res = simulate(p, n, root, oracle.skips(p), recv, send, rounds_of)
        arrival, stats = oracle.simulate_broadcast(p, root, n, recv, send)
        assert ((arrival >= 0).T == res["held"]).all()
        assert int(arrival.max()) == res["done_round"]


def test_simulated_broadcast_notices_damaged_tables():
    p, n, root = 37, 9, 4
    recv, send = oracle.schedule_table(p, root)
    q = recv.shape[1]
    # a send entry changed: the receiver no longer gets what it expects
    s2 = send.copy(); s2[10, 2] = s2[10, 2] - 1 if s2[10, 2] > -q else s2[10, 2] + 1
    arrival, stats = oracle.simulate_broadcast(p, root, n, recv, s2)
    assert stats[0] + stats[3] > 0 and stats[4] > 0 and (arrival < 0).any()
    # an entry out of range is counted and moves nothing
    r2 = recv.copy(); r2[20, 1] = q
    _, stats = oracle.simulate_broadcast(p, root, n, r2, send)
    assert stats[5] == 1 and stats[3] + stats[0] > 0
    # a processor and its from-processor agree on a block the sender does not hold yet: both tables of
    # round 0 say "block of the next phase"
    a = (root + 5) % p
    f = (a - 1) % p
    r3, s3 = recv.copy(), send.copy()
    r3[a, 0] = q - 1; s3[f, 0] = q - 1
    _, stats = oracle.simulate_broadcast(p, root, n, r3, s3)
    assert stats[1] > 0
    # the tables of another root
    _, stats = oracle.simulate_broadcast(p, (root + 1) % p, n, recv, send)
    assert sum(int(v) for v in stats[:5]) > 0


def test_shifted_tables_are_algorithm_1s_starting_rows():
    for p in [2, 9, 17, 18, 100]:
        q = oracle.q_of(p)
        recv, send = oracle.schedule_table(p)
        for n in range(1, 3 * q + 2):
            x, srecv, ssend = oracle.shifted_table(p, n)
            assert (n - 1 + x) % q == 0 and 0 <= x < q
            for a in [0, 1, p // 2, p - 1]:
                # the first use of entry k in the printed loop reads exactly the shifted entry
                _, k, rr, sr = oracle.broadcast_rounds(q, n, recv[a], send[a])
                seen = set()
                for j in range(min(n - 1 + q, q)):
                    if int(k[j]) not in seen:
                        seen.add(int(k[j]))
                        assert rr[j] == srecv[a, k[j]] and sr[j] == ssend[a, k[j]]
            # entries of rounds before x belong to the next phase
            assert ((srecv - recv) == np.where(np.arange(q) < x, q - x, -x)).all()


def _contributions(p, n, seed):
    return np.random.default_rng(seed).integers(0, 2 ** 63, size=(n, p), dtype=np.uint64)


def test_simulated_reduction_gives_the_sum():
    for p in list(range(1, 34)) + [63, 64, 65, 100]:
        q = oracle.q_of(p)
        for n in [1, 2, q, q + 1, 2 * q + 3]:
            if n < 1:
                continue
            for root in {0, p // 3, p - 1}:
                recv, send = oracle.schedule_table(p, root)
                value = _contributions(p, n, p * 131 + n)
                result, stats = oracle.simulate_reduce(p, root, n, recv, send, value)
                with np.errstate(over="ignore"):
                    want = value.sum(axis=1, dtype=np.uint64)           # the definition of the reduction
                assert (result == want).all(), (p, n, root)
                assert list(stats[:6]) == [0] * 6, (p, n, root, stats)
                assert stats[6] == (p - 1) * n                          # every partial result moved exactly once


def test_simulated_reduction_notices_damaged_tables():
    p, n, root = 37, 9, 4
    recv, send = oracle.schedule_table(p, root)
    q = recv.shape[1]
    value = _contributions(p, n, 7)
    with np.errstate(over="ignore"):
        want = value.sum(axis=1, dtype=np.uint64)
    r2 = recv.copy(); r2[10, 2] = r2[10, 2] - 1 if r2[10, 2] > -q else r2[10, 2] + 1
    result, stats = oracle.simulate_reduce(p, root, n, r2, send, value)
    assert sum(int(v) for v in stats[:5]) > 0 and (result != want).any()
    result, stats = oracle.simulate_reduce(p, (root + 1) % p, n, recv, send, value)
    assert sum(int(v) for v in stats[:5]) > 0


# ---------------------------------------------------------------- Algorithm 7 by all processors; its reversal
def test_simulated_allbroadcast_of_correct_tables():
    """Observation 1 item 2 / Algorithm 7: all p broadcasts share the rounds.  Every processor ends with all
    n blocks of every root after exactly n-1+q rounds, nothing is packed before it is held, packed and
    unpacked blocks agree root by root, and the broadcast from root j runs exactly as Algorithm 1 alone
    would run it (whose arrival rounds Theorem 1 pins)."""
    for p in list(range(1, 20)) + [33, 64, 65]:
        q = oracle.q_of(p)
        for n in sorted({1, 2, 3, max(q, 1), q + 2}):
            arrival, stats = oracle.simulate_allbroadcast(p, n)
            assert list(stats[:6]) == [0] * 6, (p, n, stats)
            assert stats[6] == (p - 1) * n * p
            if p > 1:
                assert stats[7] == n - 1 + q
            for j in range(p) if p <= 19 else (0, 1, p // 2, p - 1):
                recv, send = oracle.schedule_table(p, j)
                alone, _ = oracle.simulate_broadcast(p, j, n, recv, send)
                assert np.array_equal(arrival[j], alone), (p, n, j)
            # the same from the root-0 tables read at row (r - j) mod p
            recv0, send0 = oracle.schedule_table(p, 0)
            arrival0, stats0 = oracle.simulate_allbroadcast(p, n, recv0, send0)
            assert np.array_equal(arrival, arrival0) and list(stats) == list(stats0)


def test_simulated_allbroadcast_power_of_two_single_block():
    # p = 2^q, n = 1: processor r gets root j's block in round floor(log2((r - j) mod p)) + 1
    for q in range(1, 7):
        p = 2 ** q
        arrival, stats = oracle.simulate_allbroadcast(p, 1)
        for j in range(p):
            for r in range(p):
                v = (r - j) % p
                assert arrival[j, 0, r] == (0 if v == 0 else v.bit_length()), (p, j, r)


def test_simulated_allbroadcast_notices_damaged_tables():
    p, n = 21, 6
    q = oracle.q_of(p)
    recv0, send0 = oracle.schedule_table(p, 0)
    r2 = recv0.copy(); r2[7, 2] = q + 3                       # out of range: every (processor, root) pair with
    _, stats = oracle.simulate_allbroadcast(p, n, r2, send0)  # (r - j) mod p = 7 reads it
    assert stats[5] == p and stats[4] > 0
    s2 = send0.copy(); s2[5, 1] = s2[5, 1] - 1 if s2[5, 1] > -q else s2[5, 1] + 1
    _, stats = oracle.simulate_allbroadcast(p, n, recv0, s2)
    assert sum(int(v) for v in stats[:5]) > 0
    # tables of another p's shape would not even have the right size; tables of another root do
    recv1, send1 = oracle.schedule_table(p, 1)
    _, stats = oracle.simulate_allbroadcast(p, n, recv1, send1)
    assert sum(int(v) for v in stats[:5]) > 0


def test_simulated_allreduction_gives_every_root_its_sums():
    """Observation 1 item 4: the rounds reversed.  Root j ends with the sum over all processors of the
    contributions to each of its blocks (the definition of the reduction), every partial result of every
    non-root processor is passed on exactly once, and root j's reduction is what the reversal of
    Algorithm 1 alone gives."""
    for p in list(range(1, 20)) + [33, 64, 65]:
        q = oracle.q_of(p)
        for n in sorted({1, 2, max(q, 1), q + 2}):
            value = np.random.default_rng(p * 977 + n).integers(0, 2 ** 63, size=(p, n, p), dtype=np.uint64)
            result, stats = oracle.simulate_allreduce(p, n, value)
            with np.errstate(over="ignore"):
                want = value.sum(axis=2, dtype=np.uint64)
            assert np.array_equal(result, want), (p, n)
            assert list(stats[:6]) == [0] * 6, (p, n, stats)
            assert stats[6] == (p - 1) * n * p
            for j in (0, p // 2, p - 1):
                recv, send = oracle.schedule_table(p, j)
                alone, _ = oracle.simulate_reduce(p, j, n, recv, send, value[j])
                assert np.array_equal(result[j], alone), (p, n, j)
            recv0, send0 = oracle.schedule_table(p, 0)
            result0, stats0 = oracle.simulate_allreduce(p, n, value, recv0, send0)
            assert np.array_equal(result, result0) and list(stats) == list(stats0)


def test_simulated_allreduction_notices_damaged_tables():
    p, n = 21, 6
    q = oracle.q_of(p)
    recv0, send0 = oracle.schedule_table(p, 0)
    value = np.random.default_rng(3).integers(0, 2 ** 63, size=(p, n, p), dtype=np.uint64)
    with np.errstate(over="ignore"):
        want = value.sum(axis=2, dtype=np.uint64)
    r2 = recv0.copy(); r2[9, 1] = r2[9, 1] - 1 if r2[9, 1] > -q else r2[9, 1] + 1
    result, stats = oracle.simulate_allreduce(p, n, value, r2, send0)
    assert sum(int(v) for v in stats[:5]) > 0 and (result != want).any()
    s2 = send0.copy(); s2[3, 0] = q + 1
    _, stats = oracle.simulate_allreduce(p, n, value, recv0, s2)
    assert stats[5] == p
