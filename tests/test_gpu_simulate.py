"""GPU parity of the entry points that USE schedule tables: Algorithm 1 run by all processors
(bcast_simulate_broadcast), its reversal as a reduction (bcast_simulate_reduce), both for all p roots at
once (Algorithm 7: bcast_simulate_allbroadcast, bcast_simulate_allreduce), and the tables
with Algorithm 1's preamble applied (bcast_schedule_shifted).  All through the C ABI, bit for bit
against the CPU oracle on the same tables."""
import numpy as np
import pytest

import oracle
import paper_2407_18004_b200 as bs
from paper_2407_18004_b200 import workloads

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


@pytest.fixture(scope="module", autouse=True)
def _need_gpu():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")


@pytest.fixture(params=["launches", "fused"])
def rounds(request):
    """The single-root simulators with one launch per round, and with all rounds in cooperative launches."""
    bs.bcast_set_simulate_rounds({"launches": bs.BCAST_ROUNDS_LAUNCHES, "fused": bs.BCAST_ROUNDS_FUSED}[request.param])
    yield request.param
    bs.bcast_set_simulate_rounds(bs.BCAST_ROUNDS_AUTO)


def dev(a):
    return torch.from_numpy(np.ascontiguousarray(a)).cuda()


def u64(t):
    return t.cpu().numpy().view(np.uint64)


def check_broadcast(p, root, n, recv, send):
    """recv/send: numpy tables given to both sides."""
    want_arrival, want_stats = oracle.simulate_broadcast(p, root, n, recv, send)
    arrival, stats = bs.simulate_broadcast(p, root, n, dev(recv) if p > 1 else None, dev(send) if p > 1 else None)
    torch.cuda.synchronize()
    assert u64(stats).tolist() == want_stats.tolist()
    assert np.array_equal(arrival.cpu().numpy(), want_arrival)
    return want_stats


# ------------------------------------------------------------------ broadcast
@pytest.mark.parametrize("p", [1, 2, 3, 17, 255, 256, 257, 1000, 4099])
def test_broadcast_small_p_every_phase_offset(p, rounds):
    q = oracle.q_of(p)
    for root in sorted({0, p // 3, p - 1}):
        recv, send = oracle.schedule_table(p, root)
        for n in sorted({1, 2, max(q, 1), q + 1, 2 * q + 3, 8}):
            stats = check_broadcast(p, root, n, recv, send)
            assert stats[:6].tolist() == [0] * 6 and stats[6] == (p - 1) * n
            assert stats[7] == (n - 1 + q if p > 1 else 0)


def test_broadcast_config1_on_gpu_tables(rounds):
    # config 1: p = 1000, 8 blocks over 17 rounds, on the tables the GPU itself computed
    p, n = workloads.P_SMALL, 8
    recv, send = bs.schedule(p, 0)
    arrival, stats = bs.simulate_broadcast(p, 0, n, recv, send)
    torch.cuda.synchronize()
    want_arrival, want_stats = oracle.simulate_broadcast(p, 0, n, *oracle.schedule_table(p, 0))
    assert u64(stats).tolist() == want_stats.tolist() == [0, 0, 0, 0, 0, 0, 999 * 8, 17]
    assert np.array_equal(arrival.cpu().numpy(), want_arrival)


def test_broadcast_medium_p_many_blocks(rounds):
    # several tiles of 256 processors with a ragged tail, more blocks than one phase, other root
    p, root, n = 70001, 12345, 40
    recv, send = oracle.schedule_table(p, root)
    stats = check_broadcast(p, root, n, recv, send)
    assert stats[:6].tolist() == [0] * 6


@pytest.mark.parametrize("n", [24, 64])
def test_broadcast_config2_on_gpu_tables_properties(rounds, n):
    # config 2's p on the GPU's own tables (n = 64 is the benchmark's simulation): too large for the oracle's
    # simulation in seconds, so the facts that hold at any size are checked, and sampled processors against
    # Theorem 1 row by row
    p = workloads.P_MEDIUM
    q = bs.bcast_q(p)
    recv, send = bs.schedule(p, 0)
    arrival, stats = bs.simulate_broadcast(p, 0, n, recv, send)
    torch.cuda.synchronize()
    assert u64(stats).tolist() == [0, 0, 0, 0, 0, 0, (p - 1) * n, n - 1 + q]
    assert int(arrival.min()) == 0 and int(arrival.max()) == n - 1 + q
    assert int((arrival[:, 0] != 0).sum()) == 0 and int((arrival[:, 1:] < 1).sum()) == 0
    x = (q - (n - 1) % q) % q
    rng = np.random.default_rng(3)
    for a in [1, 2, p - 1, p // 2] + [int(v) for v in rng.integers(1, p, 12)]:
        row = oracle.recvschedule(p, a)
        col = arrival[:, a].cpu().numpy()
        for j in range(n - 1 + q):
            i = x + j
            raw = int(row[i % q]) + q * (i // q) - x
            if raw >= 0:
                assert col[min(raw, n - 1)] == j + 1


def damaged_tables(p, root, seed, count):
    """Correct tables with `count` entries changed on the host (the mistakes are planted in the inputs)."""
    recv, send = oracle.schedule_table(p, root)
    q = recv.shape[1]
    rng = np.random.default_rng(seed)
    for _ in range(count):
        tab = recv if rng.integers(2) else send
        tab[rng.integers(p), rng.integers(q)] = rng.integers(-q - 2, q + 2)
    return recv, send


@pytest.mark.parametrize("p,root,n,count", [(37, 4, 9, 1), (300, 0, 5, 6), (1000, 77, 13, 40), (5000, 1, 3, 500)])
def test_broadcast_damaged_tables_same_findings(p, root, n, count, rounds):
    recv, send = damaged_tables(p, root, p + n, count)
    stats = check_broadcast(p, root, n, recv, send)
    assert sum(int(v) for v in stats[:6]) > 0
    # tables of another root, and consistent tables that let a block travel too early
    recv, send = oracle.schedule_table(p, root)
    check_broadcast(p, (root + 1) % p, n, recv, send)
    a = (root + 5) % p
    recv[a, 0] = recv.shape[1] - 1
    send[(a - 1) % p, 0] = recv.shape[1] - 1
    stats = check_broadcast(p, root, n, recv, send)
    assert stats[1] > 0


def test_simulate_argument_errors():
    p, n = 100, 4
    recv, send = bs.schedule(p, 0)
    arrival = torch.empty((n, p), dtype=torch.int32, device="cuda")
    stats = torch.empty(8, dtype=torch.int64, device="cuda")
    scratch = torch.empty(bs.bcast_simulate_scratch_bytes(p, n), dtype=torch.uint8, device="cuda")
    for args, code in [((0, 0, n, recv, send, arrival, stats, scratch), -1),
                       ((p, p, n, recv, send, arrival, stats, scratch), -2),
                       ((p, 0, 0, recv, send, arrival, stats, scratch), -6),
                       ((p, 0, n, None, send, arrival, stats, scratch), -4),
                       ((p, 0, n, recv, send, None, stats, scratch), -4),
                       ((p, 0, n, recv, send, arrival, stats, None), -4),
                       ((p, 0, n, recv, send, arrival, stats, scratch[:64]), -10)]:
        with pytest.raises(bs.BcastError) as e:
            bs.bcast_simulate_broadcast(*args)
        assert e.value.code == code
    value = torch.zeros((n, p), dtype=torch.int64, device="cuda")
    result = torch.zeros(n, dtype=torch.int64, device="cuda")
    with pytest.raises(bs.BcastError) as e:
        bs.bcast_simulate_reduce(p, 0, n, recv, send, value, result, stats, scratch)   # broadcast-sized scratch
    assert e.value.code == -10
    torch.cuda.synchronize()


# ------------------------------------------------------------------ reduction
def contributions(p, n, seed):
    return np.random.default_rng(seed).integers(0, 2 ** 63, size=(n, p), dtype=np.uint64)


def check_reduce(p, root, n, recv, send, value):
    want_result, want_stats = oracle.simulate_reduce(p, root, n, recv, send, value)
    result, stats = bs.simulate_reduce(p, root, n, dev(recv) if p > 1 else None, dev(send) if p > 1 else None,
                                       dev(value.view(np.int64)))
    torch.cuda.synchronize()
    assert u64(stats).tolist() == want_stats.tolist()
    assert u64(result).tolist() == want_result.tolist()
    return want_result, want_stats


@pytest.mark.parametrize("p", [1, 2, 3, 17, 256, 257, 1000, 4099])
def test_reduce_small_p(p, rounds):
    q = oracle.q_of(p)
    for root in sorted({0, p // 3, p - 1}):
        recv, send = oracle.schedule_table(p, root)
        for n in sorted({1, max(q, 1), q + 1, 2 * q + 3}):
            value = contributions(p, n, p + n)
            result, stats = check_reduce(p, root, n, recv, send, value)
            with np.errstate(over="ignore"):
                assert result.tolist() == value.sum(axis=1, dtype=np.uint64).tolist()
            assert stats[:6].tolist() == [0] * 6 and stats[6] == (p - 1) * n


def test_reduce_medium_p_on_gpu_tables(rounds):
    p, root, n = 70001, 4321, 30
    recv, send = bs.schedule(p, root)
    value = contributions(p, n, 11)
    result, stats = bs.simulate_reduce(p, root, n, recv, send, dev(value.view(np.int64)))
    torch.cuda.synchronize()
    with np.errstate(over="ignore"):
        assert u64(result).tolist() == value.sum(axis=1, dtype=np.uint64).tolist()
    assert u64(stats).tolist() == [0, 0, 0, 0, 0, 0, (p - 1) * n, 0]
    orecv, osend = oracle.schedule_table(p, root)
    check_reduce(p, root, n, orecv, osend, value)


def test_reduce_config2_on_gpu_tables_sums(rounds):
    # the benchmark's reduction (config 2's p, 64 blocks) on the GPU's own tables: the root must end up with the
    # wrapping sum of every block's contributions, every partial result combined exactly once
    p, n = workloads.P_MEDIUM, 64
    recv, send = bs.schedule(p, 0)
    gen = torch.Generator(device="cuda")
    gen.manual_seed(5)
    value = torch.randint(0, 2 ** 62, (n, p), dtype=torch.int64, device="cuda", generator=gen)
    result, stats = bs.simulate_reduce(p, 0, n, recv, send, value)
    torch.cuda.synchronize()
    assert torch.equal(result, value.sum(dim=1))               # int64 sums wrap like the uint64 ones
    assert u64(stats).tolist() == [0, 0, 0, 0, 0, 0, (p - 1) * n, 0]


@pytest.mark.parametrize("p,root,n,count", [(37, 4, 9, 1), (300, 0, 5, 6), (1000, 77, 13, 40)])
def test_reduce_damaged_tables_same_findings(p, root, n, count, rounds):
    recv, send = damaged_tables(p, root, 3 * p + n, count)
    value = contributions(p, n, 5)
    _, stats = check_reduce(p, root, n, recv, send, value)
    assert sum(int(v) for v in stats[:6]) > 0
    recv, send = oracle.schedule_table(p, root)
    check_reduce(p, (root + 1) % p, n, recv, send, value)


# ------------------------------------------------------------------ shifted tables
@pytest.mark.parametrize("p,root", [(2, 0), (17, 0), (1000, 0), (1000, 999), (5000, 1234), (70001, 5)])
def test_shifted_tables(p, root):
    q = oracle.q_of(p)
    for n in sorted({1, 2, q, q + 1, q + 2, 2 * q - 1, 8, 1000}):
        x, want_recv, want_send = oracle.shifted_table(p, n, root)
        recv = torch.empty((p, q), dtype=torch.int32, device="cuda")
        send = torch.empty((p, q), dtype=torch.int32, device="cuda")
        assert bs.bcast_schedule_shifted(p, root, n, 0, p, recv, send) == q
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy(), want_recv), (p, n)
        assert np.array_equal(send.cpu().numpy(), want_send), (p, n)
        k, shift = bs.bcast_round(q, n, 0)
        assert -shift == x


def test_shifted_tables_ranges_and_unaligned():
    p, root, n = 100003, 17, 12
    q = oracle.q_of(p)
    for lo, hi in [(0, 1), (255, 513), (p - 300, p), (1000, 1000)]:
        x, want_recv, want_send = oracle.shifted_table(p, n, root, lo, hi)
        buf = torch.empty((hi - lo) * q + 1, dtype=torch.int32, device="cuda")
        recv = buf[1:].view(hi - lo, q)                    # 4-byte aligned only: the scalar store path
        send = torch.empty((hi - lo, q), dtype=torch.int32, device="cuda")
        bs.bcast_schedule_shifted(p, root, n, lo, hi, recv, send)
        torch.cuda.synchronize()
        assert np.array_equal(recv.cpu().numpy(), want_recv) and np.array_equal(send.cpu().numpy(), want_send)
    with pytest.raises(bs.BcastError) as e:
        bs.bcast_schedule_shifted(p, root, 0, 0, 1, send, send)
    assert e.value.code == -6


def test_more_blocks_than_one_launch_grid_holds(rounds):
    # n above 65535: the per-block launches (arrival set-up, the reduction's last pass) go in slices
    p, root, n = 5, 3, 70001
    recv, send = oracle.schedule_table(p, root)
    stats = check_broadcast(p, root, n, recv, send)
    assert stats[:6].tolist() == [0] * 6 and stats[6] == (p - 1) * n and stats[7] == n - 1 + 3
    value = contributions(p, n, 1)
    result, rstats = check_reduce(p, root, n, recv, send, value)
    with np.errstate(over="ignore"):
        assert result.tolist() == value.sum(axis=1, dtype=np.uint64).tolist()
    assert rstats[:6].tolist() == [0] * 6


def test_more_rounds_than_one_cooperative_launch_holds_on_several_blocks(rounds):
    # n - 1 + q above 65536 rounds on four blocks of processors: the fused form goes in two launches, and
    # the blocks' meeting counter carries over from the first to the second
    p, root, n = 1000, 7, 65600
    recv, send = oracle.schedule_table(p, root)
    stats = check_broadcast(p, root, n, recv, send)
    assert stats[:6].tolist() == [0] * 6 and stats[6] == (p - 1) * n and stats[7] == n - 1 + 10
    value = contributions(p, n, 2)
    result, rstats = check_reduce(p, root, n, recv, send, value)
    assert rstats[:6].tolist() == [0] * 6 and rstats[6] == (p - 1) * n


def test_bounded_wait_runs_out_and_says_so():
    # the blocks of the fused form are told to wait for one block more than there are: every wait gives up after
    # about two seconds, every block stops, all eight statistics words come back as all-ones, and the context
    # is as usable as before
    p, n = 3000, 4                                         # three blocks of 1024 threads, 15 rounds
    recv, send = bs.schedule(p, 0)
    value = dev(contributions(p, n, 3).view(np.int64))
    bs.bcast_set_simulate_rounds(bs.BCAST_ROUNDS_FUSED_MISS)
    try:
        _, stats = bs.simulate_broadcast(p, 0, n, recv, send)
        _, rstats = bs.simulate_reduce(p, 0, n, recv, send, value)
        torch.cuda.synchronize()
    finally:
        bs.bcast_set_simulate_rounds(bs.BCAST_ROUNDS_AUTO)
    assert u64(stats).tolist() == [2 ** 64 - 1] * 8
    assert u64(rstats).tolist() == [2 ** 64 - 1] * 8
    orecv, osend = oracle.schedule_table(p, 0)
    stats = check_broadcast(p, 0, n, orecv, osend)
    assert stats[:6].tolist() == [0] * 6 and stats[6] == (p - 1) * n


# ------------------------------------------------------------------ all roots at once: Algorithm 7 and its reversal
def check_all(p, n, recv0, send0, tables_from_algorithm7):
    """The device gets the root-0 tables; the oracle takes every processor's tables from Algorithm 7's own
    loops (correct tables) or reads the same given tables at row (r - j) mod p (damaged tables)."""
    given = (None, None) if tables_from_algorithm7 else (recv0, send0)
    want_arrival, want_stats = oracle.simulate_allbroadcast(p, n, *given)
    d_recv, d_send = (dev(recv0), dev(send0)) if p > 1 else (None, None)
    arrival, stats = bs.simulate_allbroadcast(p, n, d_recv, d_send)
    value = np.random.default_rng(p * 31 + n).integers(0, 2 ** 63, size=(p, n, p), dtype=np.uint64)
    want_result, want_rstats = oracle.simulate_allreduce(p, n, value, *given)
    result, rstats = bs.simulate_allreduce(p, n, d_recv, d_send, dev(value.view(np.int64)))
    torch.cuda.synchronize()
    assert u64(stats).tolist() == want_stats.tolist()
    assert np.array_equal(arrival.cpu().numpy(), want_arrival)
    assert u64(rstats).tolist() == want_rstats.tolist()
    assert np.array_equal(u64(result), want_result)
    return want_stats, want_rstats, value, want_result


@pytest.mark.parametrize("p", [1, 2, 3, 9, 17, 18, 64, 100, 257])
def test_allbroadcast_and_allreduction_every_phase_offset(p):
    q = oracle.q_of(p)
    recv0, send0 = oracle.schedule_table(p, 0)
    for n in sorted({1, 2, max(q, 1), q + 1, 2 * q + 3}):
        stats, rstats, value, result = check_all(p, n, recv0, send0, True)
        assert stats[:6].tolist() == [0] * 6 and stats[6] == p * (p - 1) * n
        assert rstats[:6].tolist() == [0] * 6 and rstats[6] == p * (p - 1) * n
        with np.errstate(over="ignore"):
            assert np.array_equal(result, value.sum(axis=2, dtype=np.uint64))


def test_allbroadcast_and_allreduction_on_device_tables():
    # the tables the library itself wrote, p large enough for several blocks of processors and of roots
    p, n = 1500, 5
    q = bs.bcast_q(p)
    recv, send = bs.schedule(p, 0)
    arrival, stats = bs.simulate_allbroadcast(p, n, recv, send)
    value = torch.randint(0, 2 ** 62, (p, n, p), dtype=torch.int64, device="cuda",
                          generator=torch.Generator(device="cuda").manual_seed(1))
    result, rstats = bs.simulate_allreduce(p, n, recv, send, value)
    torch.cuda.synchronize()
    assert u64(stats).tolist() == [0, 0, 0, 0, 0, 0, p * (p - 1) * n, n - 1 + q]
    assert u64(rstats).tolist() == [0, 0, 0, 0, 0, 0, p * (p - 1) * n, 0]
    assert bool((result == value.sum(dim=2)).all())
    # root j's slab is Algorithm 1 alone from root j
    for j in (0, 700, p - 1):
        orecv, osend = oracle.schedule_table(p, j)
        alone, _ = oracle.simulate_broadcast(p, j, n, orecv, osend)
        assert np.array_equal(arrival[j].cpu().numpy(), alone)


def test_allbroadcast_and_allreduction_on_damaged_tables():
    p, n = 45, 7
    q = oracle.q_of(p)
    recv0, send0 = oracle.schedule_table(p, 0)
    r2 = recv0.copy(); r2[7, 2] = q + 3
    stats, rstats, _, _ = check_all(p, n, r2, send0, False)
    assert stats[5] == p and rstats[5] == p
    s2 = send0.copy(); s2[5, 1] = s2[5, 1] - 1 if s2[5, 1] > -q else s2[5, 1] + 1
    stats, rstats, _, _ = check_all(p, n, recv0, s2, False)
    assert sum(int(v) for v in stats[:5]) > 0 and sum(int(v) for v in rstats[:5]) > 0
    recv1, send1 = oracle.schedule_table(p, 1)
    stats, _, _, _ = check_all(p, n, recv1, send1, False)
    assert sum(int(v) for v in stats[:5]) > 0


def test_allbroadcast_argument_errors():
    p, n = 17, 3
    recv, send = bs.schedule(p, 0)
    arrival = torch.empty((p, n, p), dtype=torch.int32, device="cuda")
    stats = torch.zeros(8, dtype=torch.int64, device="cuda")
    small = torch.empty(16, dtype=torch.uint8, device="cuda")
    with pytest.raises(bs.BcastError):
        bs.bcast_simulate_allbroadcast(p, n, recv, send, arrival, stats, small)
    with pytest.raises(bs.BcastError):
        bs.bcast_simulate_allbroadcast(p, 0, recv, send, arrival, stats, small)
    with pytest.raises(bs.BcastError):
        bs.bcast_simulate_allreduce(p, n, recv, send, None, None, stats, small)
