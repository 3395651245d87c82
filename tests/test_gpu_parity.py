"""GPU parity: the CUDA path, called through the C ABI, against the CPU oracle,
bit for bit, on the same seeded inputs."""

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


def gpu_tables(p, root=0, lo=0, hi=None):
    recv, send = bs.schedule(p, root, lo, hi)
    torch.cuda.synchronize()
    return recv.cpu().numpy(), send.cpu().numpy()


def assert_equal(name, got, want):
    if not np.array_equal(got, want):
        bad = np.argwhere(got != want)
        r, k = bad[0]
        raise AssertionError(f"{name}: {len(bad)} entries differ, first at row {r} round {k}: "
                             f"gpu {got[r, k]} oracle {want[r, k]}")


# ------------------------------------------------------------------ config 1: p = 1000
def test_p1000_bit_exact_and_simulated():
    p, n = workloads.P_SMALL, 8
    recv, send = gpu_tables(p)
    orecv, osend = oracle.schedule_table(p)
    assert recv.shape == (1000, 10)
    assert_equal("recvblock", recv, orecv)
    assert_equal("sendblock", send, osend)
    # the GPU tables drive an 8-block broadcast over 17 rounds, looked up with the library's own O(1) rule
    from simulate import simulate
    q = recv.shape[1]
    skip = bs.bcast_skips(p)

    def rounds_of(rrow, srow):
        ks, rr, sr = [], [], []
        for j in range(n - 1 + q):
            k, shift = bs.bcast_round(q, n, j)
            ks.append(k); rr.append(int(rrow[k]) + shift); sr.append(int(srow[k]) + shift)
        return ks, rr, sr

    res = simulate(p, n, 0, skip, recv, send, rounds_of)
    assert res["held"].all() and res["done_round"] == 17
    assert (np.delete(res["times_received"], 0, axis=0) == 1).all()


@pytest.mark.parametrize("root", [0, 1, 499, 999])
def test_p1000_roots_and_ranges(root):
    p = 1000
    orecv, osend = oracle.schedule_table(p, root)
    for lo, hi in [(0, p), (0, 1), (999, 1000), (17, 50), (32, 64), (100, 933), (3, 3)]:
        recv, send = gpu_tables(p, root, lo, hi)
        assert_equal(f"recv[{lo}:{hi}]", recv, orecv[lo:hi])
        assert_equal(f"send[{lo}:{hi}]", send, osend[lo:hi])


def test_single_table_and_unaligned_pointers():
    p = 1234
    q = bs.bcast_q(p)
    orecv, osend = oracle.schedule_table(p, 7)
    recv, _ = bs.schedule(p, 7, want_send=False)
    _, send = bs.schedule(p, 7, want_recv=False)
    assert_equal("recv only", recv.cpu().numpy(), orecv)
    assert_equal("send only", send.cpu().numpy(), osend)
    # tables that start 4, 8 and 12 bytes off a 16-byte boundary take the scalar-store path
    for off in (1, 2, 3):
        buf_r = torch.full((p * q + 8,), 77, dtype=torch.int32, device="cuda")
        buf_s = torch.full((p * q + 8,), 77, dtype=torch.int32, device="cuda")
        bs.bcast_schedule(p, 7, 0, p, buf_r[off:], buf_s[off:])
        torch.cuda.synchronize()
        assert_equal("recv unaligned", buf_r[off:off + p * q].view(p, q).cpu().numpy(), orecv)
        assert_equal("send unaligned", buf_s[off:off + p * q].view(p, q).cpu().numpy(), osend)
        assert (buf_r[:off] == 77).all() and (buf_r[off + p * q:] == 77).all()     # nothing written outside
        assert (buf_s[:off] == 77).all() and (buf_s[off + p * q:] == 77).all()


def test_small_p_exhaustive():
    for p in list(range(2, 200)) + [255, 256, 257, 511, 512, 513]:
        recv, send = gpu_tables(p)
        orecv, osend = oracle.schedule_table(p)
        assert_equal(f"recv p={p}", recv, orecv)
        assert_equal(f"send p={p}", send, osend)


def test_degenerate_sizes():
    recv, send = bs.schedule(1)
    assert tuple(recv.shape) == (1, 0) and tuple(send.shape) == (1, 0)
    recv, send = gpu_tables(2)
    assert recv.tolist() == [[-1], [0]] and send.tolist() == [[0], [-1]]
    recv, send = bs.schedule(1000, 0, 5, 5)
    assert recv.numel() == 0
    with pytest.raises(bs.BcastError):
        bs.schedule(1000, 1000)
    with pytest.raises(bs.BcastError):
        bs.schedule(1000, 0, 10, 1001)


# ------------------------------------------------------------------ config 2: p = 2^20 + 1, full tables
def test_p_2pow20_plus_1_full_tables_bit_exact():
    p = workloads.P_MEDIUM
    recv, send = gpu_tables(p)
    assert recv.shape == (p, 21) and recv.nbytes + send.nbytes == 176160936
    orecv, osend = oracle.schedule_table(p)
    assert_equal("recvblock", recv, orecv)
    assert_equal("sendblock", send, osend)


@pytest.mark.parametrize("p", [2 ** 16, 2 ** 16 + 1, 2 ** 18 - 1, 300007, 2 ** 20, 2 ** 20 - 1])
def test_other_p_full_tables(p):
    recv, send = gpu_tables(p, root=p // 3)
    orecv, osend = oracle.schedule_table(p, root=p // 3)
    assert_equal("recvblock", recv, orecv)
    assert_equal("sendblock", send, osend)


# ------------------------------------------------------------------ config 3: p = 2^27 - 1, full tables on the device
def test_p_2pow27_minus_1_full_run_sampled_and_properties():
    p = workloads.P_LARGE
    q = bs.bcast_q(p)
    assert q == 27
    free, _ = torch.cuda.mem_get_info()
    if free < 40 * 2 ** 30:
        pytest.skip("needs 40 GB of device memory")
    recv, send = bs.schedule(p)                      # one launch, as the benchmark times it
    torch.cuda.synchronize()
    assert recv.numel() * 4 + send.numel() * 4 == 28991029032
    # (a) windows of consecutive ranks against the oracle, entry by entry
    width = 2048
    for start in workloads.sample_windows(p, width, 10, seed=3):
        stop = min(start + width, p)
        orecv, osend = oracle.schedule_table(p, 0, start, stop)
        assert_equal(f"recv[{start}:{stop}]", recv[start:stop].cpu().numpy(), orecv)
        assert_equal(f"send[{start}:{stop}]", send[start:stop].cpu().numpy(), osend)
    # (b) scattered single ranks
    ranks = workloads.sample_ranks(p, 3000, seed=4)
    got_r = recv[torch.from_numpy(ranks).cuda()].cpu().numpy()
    got_s = send[torch.from_numpy(ranks).cuda()].cpu().numpy()
    for i, r in enumerate(ranks.tolist()):
        assert got_r[i].tolist() == oracle.recvschedule(p, r).tolist(), r
        assert got_s[i].tolist() == oracle.sendschedule_alg6(p, r)[0].tolist(), r
    # (c) properties over the whole table, computed with device-side tensor operations:
    #     condition 2 (hence 1) for every rank and round, one non-negative entry per row, row sums
    skip = bs.bcast_skips(p)
    for k in range(q):
        shifted = torch.roll(recv[:, k], -int(skip[k]))         # recvblock[k] of rank (r + skip[k]) mod p
        assert bool((send[:, k] == shifted).all()), f"condition 2 fails in round {k}"
        del shifted
    nonneg = (recv >= 0).sum(dim=1)
    assert int(nonneg[0]) == 0 and bool((nonneg[1:] == 1).all())
    del nonneg
    row_sum = recv.sum(dim=1, dtype=torch.int64)
    assert int(row_sum[0]) == -q * (q + 1) // 2
    assert bool((row_sum[1:] == -q * (q + 1) // 2 + q).all())     # {-1..-q} minus (b-q) plus b
    assert bool((send[1:, 0] + q == recv[1:].max(dim=1).values).all())   # sendblock[0] = b - q
    assert send[0].tolist() == list(range(q))


# ------------------------------------------------------------------ config 4: verification sweep
def test_verify_sweep_small_range_checksums_all():
    lo, hi = 1, 600
    checksum, fails = bs.verify_sweep(lo, hi)
    torch.cuda.synchronize()
    assert fails.tolist() == [0] * 8
    got = checksum.cpu().numpy().view(np.uint64)
    for p in range(lo, hi + 1):
        assert int(got[p - lo]) == oracle.checksum(p), p


def test_verify_sweep_full_range():
    lo, hi = workloads.SWEEP_RANGE
    checksum, fails = bs.verify_sweep(lo, hi)
    torch.cuda.synchronize()
    assert fails.tolist() == [0] * 8, f"device-side invariant failures: {fails.tolist()}"
    got = checksum.cpu().numpy().view(np.uint64)
    rng = np.random.default_rng(5)
    ps = sorted(set([2, 3, 1000, 4097, 32767, 32768, 32769, 65535, 65536]
                    + [int(x) for x in rng.integers(2, hi + 1, 40)]))
    for p in ps:
        assert int(got[p - lo]) == oracle.checksum(p), p


def test_verify_sweep_small_scratch_and_offsets():
    lo, hi = 1000, 1100
    need = 256 + -(-2 * bs.bcast_q(hi) * (hi + 1) // 256) * 256
    checksum = torch.zeros(hi - lo + 1, dtype=torch.int64, device="cuda")
    fails = torch.zeros(8, dtype=torch.int32, device="cuda")
    scratch = torch.empty(need, dtype=torch.uint8, device="cuda")       # room for one block only
    bs.bcast_verify_sweep(lo, hi, checksum, fails, scratch)
    torch.cuda.synchronize()
    assert fails.tolist() == [0] * 8
    got = checksum.cpu().numpy().view(np.uint64)
    for p in (1000, 1024, 1025, 1100):
        assert int(got[p - lo]) == oracle.checksum(p)
    with pytest.raises(bs.BcastError):
        bs.bcast_verify_sweep(lo, hi, checksum, fails, scratch[:need - 256])


# ------------------------------------------------------------------ config 5: random query batch
def test_query_batch_full_size_sampled():
    nq = workloads.N_QUERIES
    p, rank, root = workloads.query_batch(nq, seed=0)
    dp, dr, do = (torch.from_numpy(x).cuda() for x in (p, rank, root))
    recv, send, bad = bs.schedule_batch(dp, dr, do, 31)
    torch.cuda.synchronize()
    assert int(bad) == 0
    rng = np.random.default_rng(6)
    pick = np.unique(np.concatenate([np.arange(64), np.arange(nq - 64, nq), rng.integers(0, nq, 6000),
                                     np.argsort(p)[-200:], np.argsort(p)[:200]]))
    idx = torch.from_numpy(pick).cuda()
    got_r, got_s = recv[idx].cpu().numpy(), send[idx].cpu().numpy()
    want_r, want_s = oracle.schedule_batch(p[pick], rank[pick], root[pick], 31)
    assert_equal("batch recv", got_r, want_r)
    assert_equal("batch send", got_s, want_s)
    # every row: q_i real entries then padding
    qs = torch.from_numpy(np.ceil(np.log2(p.astype(np.float64))).astype(np.int64)).cuda()
    col = torch.arange(31, device="cuda")[None, :]
    is_pad = col >= qs[:, None]
    assert bool(((recv == bs.BCAST_PAD) == is_pad).all()) and bool(((send == bs.BCAST_PAD) == is_pad).all())


def test_query_batch_edges():
    p = np.array([1, 2, 3, 17, 0, 10, 10, 10, 2 ** 31 - 1, 2 ** 31 - 1, -5] + [1000] * 40, dtype=np.int32)
    rank = np.array([0, 1, 2, 3, 0, 10, -1, 3, 0, 2 ** 31 - 2, 0] + list(range(40)), dtype=np.int32)
    root = np.array([0, 0, 1, 5, 0, 0, 0, 10, 2 ** 31 - 2, 5, 0] + [999] * 40, dtype=np.int32)
    good = np.array([1, 1, 1, 1, 0, 0, 0, 0, 1, 1, 0] + [1] * 40, dtype=bool)
    dp, dr, do = (torch.from_numpy(x).cuda() for x in (p, rank, root))
    for stride in (31, 32, 33, 40):
        recv = torch.full((len(p), stride), 55, dtype=torch.int32, device="cuda")
        send = torch.full((len(p), stride), 55, dtype=torch.int32, device="cuda")
        bad = torch.zeros(1, dtype=torch.int32, device="cuda")
        bs.bcast_schedule_batch(dp, dr, do, stride, recv, send, bad)
        torch.cuda.synchronize()
        assert int(bad) == int((~good).sum())
        want_r, want_s = oracle.schedule_batch(p[good], rank[good], root[good], stride)
        assert_equal("edge recv", recv.cpu().numpy()[good], want_r)
        assert_equal("edge send", send.cpu().numpy()[good], want_s)
        assert bool((recv[torch.from_numpy(~good).cuda()] == bs.BCAST_PAD).all())
        assert bool((send[torch.from_numpy(~good).cuda()] == bs.BCAST_PAD).all())
    recv_only = torch.empty((len(p), 31), dtype=torch.int32, device="cuda")
    bs.bcast_schedule_batch(dp, dr, do, 31, recv_only, None)
    torch.cuda.synchronize()
    assert_equal("recv only", recv_only.cpu().numpy()[good], oracle.schedule_batch(p[good], rank[good], root[good], 31)[0])


# ------------------------------------------------------------------ host-output entry point
def test_schedule_host_chunks():
    p, root = 100003, 17
    q = bs.bcast_q(p)
    orecv, osend = oracle.schedule_table(p, root)
    staging = torch.empty(1 << 20, dtype=torch.uint8, device="cuda")     # forces many chunks
    recv = torch.empty((p, q), dtype=torch.int32).pin_memory()
    send = torch.empty((p, q), dtype=torch.int32).pin_memory()
    bs.bcast_schedule_host(p, root, 0, p, recv, send, staging)
    torch.cuda.synchronize()
    assert_equal("host recv", recv.numpy(), orecv)
    assert_equal("host send", send.numpy(), osend)
    part = torch.empty((5000, q), dtype=torch.int32).pin_memory()
    bs.bcast_schedule_host(p, root, 777, 5777, None, part, staging)
    torch.cuda.synchronize()
    assert_equal("host send part", part.numpy(), osend[777:5777])
    with pytest.raises(bs.BcastError):
        bs.bcast_schedule_host(p, root, 0, p, recv, send, staging[:1024])


# ------------------------------------------------------------------ Algorithm 7: all-broadcast tables
@pytest.mark.parametrize("p,rank", [(2, 1), (17, 5), (1000, 0), (1000, 999), (1000, 417), (5000, 1234),
                                    (70001, 69999), (2 ** 16 + 1, 3), (2 ** 17 - 1, 77)])
@pytest.mark.parametrize("shape", ["auto", "block", "warps", "lowframe", "tight"])
def test_allbroadcast_tables(forced_shape, shape, p, rank):
    forced_shape(shape)                                        # every launch shape of the table kernel
    orecv, osend = oracle.allbroadcast_schedule(p, rank)
    recv, send = bs.allbroadcast_schedule(p, rank)
    torch.cuda.synchronize()
    assert_equal("recvblocks", recv.cpu().numpy(), orecv)
    assert_equal("sendblocks", send.cpu().numpy(), osend)
    for lo, hi in [(0, 1), (p - 1, p), (p // 3, min(p, p // 3 + 300)), (1, 1)]:
        recv, send = bs.allbroadcast_schedule(p, rank, lo, hi)
        torch.cuda.synchronize()
        assert_equal(f"recvblocks[{lo}:{hi}]", recv.cpu().numpy(), orecv[lo:hi])
        assert_equal(f"sendblocks[{lo}:{hi}]", send.cpu().numpy(), osend[lo:hi])


def test_allbroadcast_large_p_is_the_reversed_broadcast_table(forced_shape):
    """p = 2^20+1: row j of processor r's tables is row (r - j) mod p of the root-0 tables."""
    p, rank = workloads.P_MEDIUM, 777777
    recv0, send0 = bs.schedule(p)
    recv, send = bs.allbroadcast_schedule(p, rank)
    for shape in ("warps", "block", "tight"):              # the other shapes too (queues overflow in the last)
        forced_shape(shape)
        recv_w, send_w = bs.allbroadcast_schedule(p, rank)
        assert bool((recv_w == recv).all()) and bool((send_w == send).all()), shape
    torch.cuda.synchronize()
    idx = (rank - torch.arange(p, device="cuda")) % p
    assert bool((recv == recv0[idx]).all()) and bool((send == send0[idx]).all())
    # and a window against the oracle, entry by entry
    lo, hi = 500000, 501000
    orecv, osend = oracle.allbroadcast_schedule(p, rank, lo, hi)
    assert_equal("recvblocks", recv[lo:hi].cpu().numpy(), orecv)
    assert_equal("sendblocks", send[lo:hi].cpu().numpy(), osend)
    with pytest.raises(bs.BcastError):
        bs.allbroadcast_schedule(p, p)


# ------------------------------------------------------------------ largest sizes: q = 30 and 31 (64-bit walk)
@pytest.mark.parametrize("p", [2 ** 31 - 1, 2 ** 30 + 1, 2 ** 30, 2 ** 31 - 5, 1431655765])
def test_rank_windows_of_the_largest_p(p):
    """Windows of ranks of p near 2^31, where p + r passes 2^31: both ends, around skips, a wrap past
    the root, and random places; every window spans several tiles and ends ragged."""
    q = bs.bcast_q(p)
    skips = bs.bcast_skips(p)
    rng = np.random.default_rng(p % 1000)
    root = int(rng.integers(0, p))
    starts = [0, p - 1500, root - 700 if root >= 700 else 0, int(skips[q - 1]) - 600, int(skips[q - 2]) + root - 300]
    starts += [int(x) for x in rng.integers(0, p - 2000, 3)]
    for lo in starts:
        lo = max(0, min(lo, p - 1500))
        hi = lo + 1500 - (lo % 7)
        recv, send = bs.schedule(p, root, lo, hi)
        torch.cuda.synchronize()
        orecv, osend = oracle.schedule_table(p, root, lo, hi)
        assert_equal(f"p={p} recv[{lo}:{hi}]", recv.cpu().numpy(), orecv)
        assert_equal(f"p={p} send[{lo}:{hi}]", send.cpu().numpy(), osend)
    lo = p - 3000
    arecv, asend = bs.allbroadcast_schedule(p, root, lo, p)
    torch.cuda.synchronize()
    oarecv, oasend = oracle.allbroadcast_schedule(p, root, lo, p)
    assert_equal("allbroadcast recv", arecv.cpu().numpy(), oarecv)
    assert_equal("allbroadcast send", asend.cpu().numpy(), oasend)


# ------------------------------------------------------------------ tiles that cannot share their high levels
@pytest.mark.parametrize("p", [100003, 2 ** 17 + 1, 2 ** 17 - 1])
def test_windows_roots_and_single_tables_mid_p(p):
    """q = 17, 18: full tiles take the shared run descriptions; the windows below also produce tiles
    that hold the root, wrap past p-1, start off a multiple of 256 and end ragged, and launches that
    want only one of the two tables (no in-tile copies of receive entries then)."""
    q = bs.bcast_q(p)
    for root in (0, 1, 255, 256, 50000, p - 1):
        orecv, osend = oracle.schedule_table(p, root)
        for lo, hi in [(0, p), (1, 4099), (root, min(p, root + 777)), (max(0, root - 300), min(p, root + 300)),
                       (p - 1000, p), (12345, 12345 + 2048)]:
            recv, send = bs.schedule(p, root, lo, hi)
            torch.cuda.synchronize()
            assert_equal(f"root {root} recv[{lo}:{hi}]", recv.cpu().numpy(), orecv[lo:hi])
            assert_equal(f"root {root} send[{lo}:{hi}]", send.cpu().numpy(), osend[lo:hi])
        recv, _ = bs.schedule(p, root, 3, p - 5, want_send=False)
        _, send = bs.schedule(p, root, 3, p - 5, want_recv=False)
        torch.cuda.synchronize()
        assert_equal("recv only", recv.cpu().numpy(), orecv[3:p - 5])
        assert_equal("send only", send.cpu().numpy(), osend[3:p - 5])
        assert recv.shape == (p - 8, q)


# ------------------------------------------------------------------ two device implementations against each other
@pytest.mark.parametrize("p,root", [(2 ** 24 + 3, 0), (2 ** 24 + 3, 9999999), (123456789, 1), (2 ** 27 - 1, 5)])
def test_table_kernel_against_batch_kernel_at_scale(p, root):
    """Every entry of 2^24 consecutive ranks: the table kernel (closed forms, shared high levels, queues)
    against the batch kernel (search of Algorithms 4/5 and Algorithm 6 per thread).  Both are compared
    with the oracle elsewhere; here they must agree with each other where the oracle is too slow."""
    free, _ = torch.cuda.mem_get_info()
    if free < 12 * 2 ** 30:
        pytest.skip("needs 12 GB of device memory")
    n = min(p, 2 ** 24)
    q = bs.bcast_q(p)
    lo = (p - n) // 2
    recv, send = bs.schedule(p, root, lo, lo + n)
    ranks = torch.arange(lo, lo + n, dtype=torch.int32, device="cuda")
    ps = torch.full((n,), p, dtype=torch.int32, device="cuda")
    roots = torch.full((n,), root, dtype=torch.int32, device="cuda")
    brecv, bsend, bad = bs.schedule_batch(ps, ranks, roots, 31)
    torch.cuda.synchronize()
    assert int(bad) == 0
    assert bool((recv == brecv[:, :q]).all()), "receive tables differ"
    assert bool((send == bsend[:, :q]).all()), "send tables differ"


# ------------------------------------------------------------------ both launch shapes of the table kernel
@pytest.mark.parametrize("shape", ["block", "warps", "lowframe", "tight"])
@pytest.mark.parametrize("p,root", [(1000, 0), (5000, 1234), (2 ** 16 + 1, 7), (300007, 299999), (2 ** 20 + 1, 0),
                                    (2 ** 20 - 1, 5), (3 * 2 ** 18, 11), (999983, 500000)])
def test_every_launch_shape_full_tables(forced_shape, shape, p, root):
    """The library picks the launch shape from an estimate; forced each way, on p with many and with few
    undecided entries, the tables equal the oracle's.  The tight shape has next to no queue space, so every
    group of tiles with undecided entries takes the path that recomputes its rows by the search alone."""
    forced_shape(shape)
    recv, send = gpu_tables(p, root)
    orecv, osend = oracle.schedule_table(p, root)
    assert_equal("recvblock (%s)" % shape, recv, orecv)
    assert_equal("sendblock (%s)" % shape, send, osend)
    # a ragged window that starts inside a warp's slice, and single tables
    lo, hi = 37, min(p, 37 + 3 * 256 + 5)
    r2, _ = bs.schedule(p, root, lo, hi, want_send=False)
    _, s2 = bs.schedule(p, root, lo, hi, want_recv=False)
    torch.cuda.synchronize()
    assert_equal("recv window (%s)" % shape, r2.cpu().numpy(), orecv[lo:hi])
    assert_equal("send window (%s)" % shape, s2.cpu().numpy(), osend[lo:hi])
