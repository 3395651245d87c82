"""CPU oracle for the broadcast-schedule computation -- TEST INFRASTRUCTURE.

A ctypes front end for ``bcast_oracle.c`` (plain C, single-threaded, written
from the paper; see that file's header).  Nothing in the CUDA library or its
Python binding may import this package; only the tests, the smoke check and the
benchmark's CPU-baseline leg do.  This package in turn imports nothing from the
CUDA side.
"""
from __future__ import annotations

import ctypes
import os
import subprocess
import threading

import numpy as np

_HERE = os.path.dirname(os.path.abspath(__file__))
_SRC = os.path.join(_HERE, "bcast_oracle.c")
_LIB = os.path.join(_HERE, "liboracle.so")
_lock = threading.Lock()
_lib = None

PAD = -(2 ** 31)


def build(force: bool = False) -> str:
    """Compile the C oracle with gcc (no optimisation tricks, no threads)."""
    if force or not os.path.exists(_LIB) or os.path.getmtime(_LIB) < os.path.getmtime(_SRC):
        tmp = _LIB + ".tmp.%d" % os.getpid()
        subprocess.check_call(["gcc", "-O2", "-std=c99", "-Wall", "-Wextra", "-shared", "-fPIC",
                               "-o", tmp, _SRC])
        os.replace(tmp, _LIB)
    return _LIB


def _load():
    global _lib
    with _lock:
        if _lib is None:
            # ORACLE_LIBRARY: a deliberately broken build, used only by the test that checks that the
            # pins notice planted mistakes
            lib = ctypes.CDLL(os.environ.get("ORACLE_LIBRARY") or build())
            i32p = ctypes.POINTER(ctypes.c_int32)
            i64p = ctypes.POINTER(ctypes.c_int64)
            u64p = ctypes.POINTER(ctypes.c_uint64)
            i64 = ctypes.c_int64
            lib.oracle_q.argtypes = [i64]
            lib.oracle_skips.argtypes = [i64, i64p]
            lib.oracle_baseblock.argtypes = [i64, i64]
            lib.oracle_recvschedule.argtypes = [i64, i64, i32p, i64p]
            lib.oracle_recv_positions.argtypes = [i64, i64, i64p]
            lib.oracle_sendschedule_def.argtypes = [i64, i64, i32p]
            lib.oracle_sendschedule_alg6.argtypes = [i64, i64, i32p, i32p, u64p]
            lib.oracle_schedule_table.argtypes = [i64, i64, i64, i64, i32p, i32p]
            lib.oracle_allbroadcast_schedule.argtypes = [i64, i64, i64, i64, i32p, i32p]
            lib.oracle_round_k.argtypes = [ctypes.c_int, i64, i64]
            lib.oracle_round_block.argtypes = [ctypes.c_int, i64, i64, i32p]
            lib.oracle_round_block.restype = i64
            lib.oracle_broadcast_rounds.argtypes = [ctypes.c_int, i64, i32p, i32p, i32p, i64p, i64p]
            lib.oracle_checksum.argtypes = [i64, u64p]
            lib.oracle_schedule_batch.argtypes = [i32p, i32p, i32p, i64, ctypes.c_int32,
                                                  ctypes.c_int32, i32p, i32p]
            lib.oracle_sendschedule_alg6_batch.argtypes = [i32p, i32p, i32p, i64, ctypes.c_int32,
                                                           ctypes.c_int32, i32p]
            lib.oracle_shift_rows.argtypes = [ctypes.c_int, i64, i64, i32p]
            lib.oracle_simulate_broadcast.argtypes = [i64, i64, i64, i32p, i32p, i32p, u64p]
            lib.oracle_simulate_reduce.argtypes = [i64, i64, i64, i32p, i32p, u64p, u64p, u64p]
            lib.oracle_simulate_allbroadcast.argtypes = [i64, i64, i32p, i32p, i32p, u64p]
            lib.oracle_simulate_allreduce.argtypes = [i64, i64, i32p, i32p, u64p, u64p, u64p]
            _lib = lib
    return _lib


def _i32(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int32))


def _i64(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_int64))


def q_of(p: int) -> int:
    q = _load().oracle_q(p)
    if q < 0:
        raise ValueError("p must be >= 1")
    return q


def skips(p: int) -> np.ndarray:
    """Algorithm 2: skip[0..q] as int64."""
    q = q_of(p)
    out = np.zeros(q + 1, dtype=np.int64)
    _load().oracle_skips(p, _i64(out))
    return out


def baseblock(p: int, r: int) -> int:
    b = _load().oracle_baseblock(p, r)
    if b < 0:
        raise ValueError("bad (p, r)")
    return b


def recvschedule(p: int, r: int, with_stats: bool = False):
    """Algorithm 5 for virtual rank r; optionally the Lemma 5/6 counters."""
    q = q_of(p)
    out = np.zeros(max(q, 1), dtype=np.int32)
    st = np.zeros(5, dtype=np.int64)
    if _load().oracle_recvschedule(p, r, _i32(out), _i64(st)) < 0:
        raise ValueError("bad (p, r)")
    out = out[:q]
    if with_stats:
        return out, dict(calls=int(st[0]), iters=int(st[1]), retests=int(st[2]),
                         retest_hits=int(st[3]), oob=int(st[4]))
    return out


def recv_positions(p: int, r: int) -> np.ndarray:
    """The processors r'_k of Lemma 4 (numbered in [p, 2p)) behind each receive entry of r."""
    q = q_of(p)
    out = np.zeros(max(q, 1), dtype=np.int64)
    if _load().oracle_recv_positions(p, r, _i64(out)) < 0:
        raise ValueError("bad (p, r)")
    return out[:q]


def sendschedule(p: int, r: int) -> np.ndarray:
    """Send schedule by definition (q receive schedules)."""
    q = q_of(p)
    out = np.zeros(max(q, 1), dtype=np.int32)
    if _load().oracle_sendschedule_def(p, r, _i32(out)) < 0:
        raise ValueError("bad (p, r)")
    return out[:q]


def sendschedule_alg6(p: int, r: int):
    """Algorithm 6 (second routine): (row, violations, violation-round mask)."""
    q = q_of(p)
    out = np.zeros(max(q, 1), dtype=np.int32)
    v = ctypes.c_int32(0)
    m = ctypes.c_uint64(0)
    if _load().oracle_sendschedule_alg6(p, r, _i32(out), ctypes.byref(v), ctypes.byref(m)) < 0:
        raise ValueError("bad (p, r)")
    return out[:q], int(v.value), int(m.value)


def schedule_table(p: int, root: int = 0, rank_begin: int = 0, rank_end: int | None = None,
                   want_recv: bool = True, want_send: bool = True):
    """(recvblock, sendblock) int32 tables [rank_end-rank_begin, q] for actual ranks."""
    if rank_end is None:
        rank_end = p
    q = q_of(p)
    n = rank_end - rank_begin
    recv = np.zeros((max(n, 0), q), dtype=np.int32) if want_recv else None
    send = np.zeros((max(n, 0), q), dtype=np.int32) if want_send else None
    rc = _load().oracle_schedule_table(p, root, rank_begin, rank_end,
                                       _i32(recv) if want_recv else None,
                                       _i32(send) if want_send else None)
    if rc < 0:
        raise ValueError("bad arguments to schedule_table (%d)" % rc)
    return recv, send


def allbroadcast_schedule(p: int, r: int, root_begin: int = 0, root_end: int | None = None):
    """Algorithm 7's (recvblocks, sendblocks) of processor r: row j-root_begin is for root j."""
    if root_end is None:
        root_end = p
    q = q_of(p)
    n = max(root_end - root_begin, 0)
    recv = np.zeros((n, q), dtype=np.int32)
    send = np.zeros((n, q), dtype=np.int32)
    if _load().oracle_allbroadcast_schedule(p, r, root_begin, root_end, _i32(recv), _i32(send)) < 0:
        raise ValueError("bad arguments to allbroadcast_schedule")
    return recv, send


def round_k(q: int, n: int, j: int) -> int:
    return _load().oracle_round_k(q, n, j)


def round_block(q: int, n: int, j: int, row) -> int:
    """Block moved in communication round j for a schedule row: -1 none, -2 bad args."""
    row = np.ascontiguousarray(row, dtype=np.int32)
    return int(_load().oracle_round_block(q, n, j, _i32(row)))


def broadcast_rounds(q: int, n: int, recvrow, sendrow):
    """Algorithm 1 as printed for one processor: (x, k[], raw recv[], raw send[])."""
    recvrow = np.ascontiguousarray(recvrow, dtype=np.int32)
    sendrow = np.ascontiguousarray(sendrow, dtype=np.int32)
    rounds = n - 1 + q
    k = np.zeros(rounds, dtype=np.int32)
    rr = np.zeros(rounds, dtype=np.int64)
    sr = np.zeros(rounds, dtype=np.int64)
    x = _load().oracle_broadcast_rounds(q, n, _i32(recvrow), _i32(sendrow), _i32(k), _i64(rr), _i64(sr))
    if x < 0:
        raise ValueError("bad arguments")
    return x, k, rr, sr


def checksum(p: int) -> int:
    """Order-independent 64-bit checksum of the full schedule of p (root 0)."""
    c = ctypes.c_uint64(0)
    if _load().oracle_checksum(p, ctypes.byref(c)) < 0:
        raise ValueError("bad p")
    return int(c.value)


def schedule_batch(p, rank, root, row_stride: int = 31, pad: int = PAD,
                   want_recv: bool = True, want_send: bool = True):
    """Independent (p, rank, root) queries, rows padded to row_stride with pad."""
    p = np.ascontiguousarray(p, dtype=np.int32)
    rank = np.ascontiguousarray(rank, dtype=np.int32)
    root = np.ascontiguousarray(root, dtype=np.int32)
    nq = p.shape[0]
    recv = np.zeros((nq, row_stride), dtype=np.int32) if want_recv else None
    send = np.zeros((nq, row_stride), dtype=np.int32) if want_send else None
    rc = _load().oracle_schedule_batch(_i32(p), _i32(rank), _i32(root), nq, row_stride, pad,
                                       _i32(recv) if want_recv else None,
                                       _i32(send) if want_send else None)
    if rc < 0:
        raise ValueError("bad query in batch")
    return recv, send


def sendschedule_alg6_batch(p, rank, root, row_stride: int = 31, pad: int = PAD) -> np.ndarray:
    """Send rows of independent queries by Algorithm 6 (second routine), padded to row_stride."""
    p = np.ascontiguousarray(p, dtype=np.int32)
    rank = np.ascontiguousarray(rank, dtype=np.int32)
    root = np.ascontiguousarray(root, dtype=np.int32)
    nq = p.shape[0]
    send = np.zeros((nq, row_stride), dtype=np.int32)
    if _load().oracle_sendschedule_alg6_batch(_i32(p), _i32(rank), _i32(root), nq, row_stride, pad, _i32(send)) < 0:
        raise ValueError("bad query in batch")
    return send


def _u64(a):
    return a.ctypes.data_as(ctypes.POINTER(ctypes.c_uint64))


def shifted_table(p: int, n: int, root: int = 0, rank_begin: int = 0, rank_end: int | None = None):
    """Algorithm 1's preamble applied to the tables: (x, recv, send) ready for n blocks."""
    recv, send = schedule_table(p, root, rank_begin, rank_end)
    q = q_of(p)
    x = 0
    if q > 0:
        x = _load().oracle_shift_rows(q, n, recv.shape[0], _i32(recv))
        _load().oracle_shift_rows(q, n, send.shape[0], _i32(send))
        if x < 0:
            raise ValueError("bad arguments")
    return x, recv, send


def simulate_broadcast(p: int, root: int, n: int, recv_tab, send_tab):
    """Algorithm 1 by all processors on the given tables: (arrival[n][p] int32, stats[8] uint64)."""
    q = q_of(p)
    recv_tab = np.ascontiguousarray(recv_tab, dtype=np.int32).reshape(p, q)
    send_tab = np.ascontiguousarray(send_tab, dtype=np.int32).reshape(p, q)
    arrival = np.zeros((n, p), dtype=np.int32)
    stats = np.zeros(8, dtype=np.uint64)
    if _load().oracle_simulate_broadcast(p, root, n, _i32(recv_tab), _i32(send_tab), _i32(arrival),
                                         _u64(stats)) < 0:
        raise ValueError("bad arguments to simulate_broadcast")
    return arrival, stats


def simulate_reduce(p: int, root: int, n: int, recv_tab, send_tab, value):
    """Observation 1.3's reduction (wrapping 64-bit sum) on the given tables.

    value: [n][p] uint64 contributions (not modified).  Returns (result[n] uint64, stats[8] uint64).
    """
    q = q_of(p)
    recv_tab = np.ascontiguousarray(recv_tab, dtype=np.int32).reshape(p, q)
    send_tab = np.ascontiguousarray(send_tab, dtype=np.int32).reshape(p, q)
    work = np.array(value, dtype=np.uint64, copy=True).reshape(n, p)
    result = np.zeros(n, dtype=np.uint64)
    stats = np.zeros(8, dtype=np.uint64)
    if _load().oracle_simulate_reduce(p, root, n, _i32(recv_tab), _i32(send_tab), _u64(work), _u64(result),
                                      _u64(stats)) < 0:
        raise ValueError("bad arguments to simulate_reduce")
    return result, stats


def simulate_allbroadcast(p: int, n: int, recv0=None, send0=None):
    """Algorithm 7 by all processors: (arrival[p roots][n][p] int32, stats[8] uint64).

    recv0/send0 None: every processor's tables by Algorithm 7's own loops; else the root-0 broadcast
    tables [p][q] whose row (r - j) mod p serves processor r for root j (for damaged tables).
    """
    q = q_of(p)
    given = recv0 is not None and send0 is not None
    if given:
        recv0 = np.ascontiguousarray(recv0, dtype=np.int32).reshape(p, q)
        send0 = np.ascontiguousarray(send0, dtype=np.int32).reshape(p, q)
    arrival = np.zeros((p, n, p), dtype=np.int32)
    stats = np.zeros(8, dtype=np.uint64)
    if _load().oracle_simulate_allbroadcast(p, n, _i32(recv0) if given else None, _i32(send0) if given else None,
                                            _i32(arrival), _u64(stats)) < 0:
        raise ValueError("bad arguments to simulate_allbroadcast")
    return arrival, stats


def simulate_allreduce(p: int, n: int, value, recv0=None, send0=None):
    """Observation 1.4's all-reduction (wrapping 64-bit sum): value [p roots][n][p] uint64 contributions
    (not modified).  Returns (result[p][n] uint64, stats[8] uint64).  Tables as for simulate_allbroadcast."""
    q = q_of(p)
    given = recv0 is not None and send0 is not None
    if given:
        recv0 = np.ascontiguousarray(recv0, dtype=np.int32).reshape(p, q)
        send0 = np.ascontiguousarray(send0, dtype=np.int32).reshape(p, q)
    work = np.array(value, dtype=np.uint64, copy=True).reshape(p, n, p)
    result = np.zeros((p, n), dtype=np.uint64)
    stats = np.zeros(8, dtype=np.uint64)
    if _load().oracle_simulate_allreduce(p, n, _i32(recv0) if given else None, _i32(send0) if given else None,
                                         _u64(work), _u64(result), _u64(stats)) < 0:
        raise ValueError("bad arguments to simulate_allreduce")
    return result, stats
