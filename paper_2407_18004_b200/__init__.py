"""Python binding of the broadcast-schedule CUDA library (arXiv 2407.18004).

A thin ctypes layer over ``libbcast_sched.so``: the functions carry the names of
the C entry points in ``include/bcast_sched.h`` and only marshal arguments.
PyTorch is used for device memory and streams; every step of the computation
runs in the library's CUDA kernels.  There is no CPU fallback: if the library is
missing it is built with nvcc, and if that fails the import error is raised.
"""
from __future__ import annotations

import ctypes

import numpy as np

from . import build as _build

BCAST_NONE = -1
BCAST_PAD = -(2 ** 31)
BCAST_MAX_Q = 31
BCAST_STATIC_SWEEP_MAX_P = 65536
BCAST_UNRESOLVED = -128
BCAST_SHAPE_AUTO, BCAST_SHAPE_BLOCK, BCAST_SHAPE_WARPS, BCAST_SHAPE_LOWFRAME, BCAST_SHAPE_WARPS_TIGHT = -1, 0, 1, 2, 3
BCAST_ROUNDS_AUTO, BCAST_ROUNDS_LAUNCHES, BCAST_ROUNDS_FUSED, BCAST_ROUNDS_FUSED_MISS = 0, 1, 2, 3

_lib = None


class BcastError(RuntimeError):
    def __init__(self, code: int):
        self.code = code
        super().__init__("bcast_sched error %d: %s" % (code, bcast_strerror(code)))


def _load():
    global _lib
    if _lib is None:
        path = _build.build()
        lib = ctypes.CDLL(path)
        i32, i64, vp = ctypes.c_int32, ctypes.c_int64, ctypes.c_void_p
        lib.bcast_strerror.argtypes = [ctypes.c_int]
        lib.bcast_strerror.restype = ctypes.c_char_p
        lib.bcast_q.argtypes = [i32]
        lib.bcast_set_launch_shape.argtypes = [ctypes.c_int]
        lib.bcast_set_simulate_rounds.argtypes = [ctypes.c_int]
        lib.bcast_skips.argtypes = [i32, vp]
        lib.bcast_schedule.argtypes = [i32, i32, i64, i64, vp, vp, vp]
        lib.bcast_schedule_host.argtypes = [i32, i32, i64, i64, vp, vp, vp, i64, vp]
        lib.bcast_allbroadcast_schedule.argtypes = [i32, i32, i64, i64, vp, vp, vp]
        lib.bcast_schedule_batch.argtypes = [vp, vp, vp, i64, i32, vp, vp, vp, vp]
        lib.bcast_verify_sweep_scratch_bytes.argtypes = [i32, i32]
        lib.bcast_verify_sweep_scratch_bytes.restype = i64
        lib.bcast_verify_sweep.argtypes = [i32, i32, vp, vp, vp, i64, vp]
        lib.bcast_verify_sweep_static.argtypes = [i32, i32, vp, vp, vp]
        lib.bcast_schedule_shifted.argtypes = [i32, i32, i64, i64, i64, vp, vp, vp]
        lib.bcast_simulate_scratch_bytes.argtypes = [i32, i64, ctypes.c_int]
        lib.bcast_simulate_scratch_bytes.restype = i64
        lib.bcast_simulate_broadcast.argtypes = [i32, i32, i64, vp, vp, vp, vp, vp, i64, vp]
        lib.bcast_simulate_reduce.argtypes = [i32, i32, i64, vp, vp, vp, vp, vp, vp, i64, vp]
        lib.bcast_store_ceiling.argtypes = [vp, i64, i64, vp]
        lib.bcast_low_states.argtypes = [i32, vp, i32]
        lib.bcast_simulate_all_scratch_bytes.argtypes = [i32, i64, ctypes.c_int]
        lib.bcast_simulate_all_scratch_bytes.restype = i64
        lib.bcast_simulate_allbroadcast.argtypes = [i32, i64, vp, vp, vp, vp, vp, i64, vp]
        lib.bcast_simulate_allreduce.argtypes = [i32, i64, vp, vp, vp, vp, vp, vp, i64, vp]
        lib.bcast_round.argtypes = [i32, i64, i64, ctypes.POINTER(i32), ctypes.POINTER(i64)]
        lib.bcast_round_block.argtypes = [i32, i64, i64, vp]
        lib.bcast_round_block.restype = i64
        _lib = lib
    return _lib


def library_path() -> str:
    _load()
    return _build.LIBRARY


def _check(rc: int) -> int:
    if rc < 0:
        raise BcastError(int(rc))
    return int(rc)


def _ptr(t):
    """Device (or host) address of a tensor / numpy array, None -> NULL."""
    if t is None:
        return None
    if isinstance(t, np.ndarray):
        return t.ctypes.data
    return t.data_ptr()


def _stream(stream):
    if stream is None:
        import torch
        return torch.cuda.current_stream().cuda_stream
    return getattr(stream, "cuda_stream", stream)


# ------------------------------------------------------------------ host-only entry points
def bcast_strerror(code: int) -> str:
    return _load().bcast_strerror(code).decode()


def bcast_set_launch_shape(shape: int) -> int:
    return _check(_load().bcast_set_launch_shape(shape))


def bcast_set_simulate_rounds(mode: int) -> int:
    return _check(_load().bcast_set_simulate_rounds(mode))


def bcast_q(p: int) -> int:
    return _check(_load().bcast_q(p))


def bcast_skips(p: int) -> np.ndarray:
    q = bcast_q(p)
    out = np.zeros(q + 1, dtype=np.int32)
    _check(_load().bcast_skips(p, out.ctypes.data))
    return out


def bcast_store_ceiling(buffer, nbytes: int, bytes_per_block: int = 0, stream=None) -> int:
    return _check(_load().bcast_store_ceiling(_ptr(buffer), nbytes, bytes_per_block, _stream(stream)))


def bcast_low_states(p: int, capacity: int = 512) -> np.ndarray:
    out = np.zeros(capacity, dtype=np.uint32)
    count = _check(_load().bcast_low_states(p, out.ctypes.data, capacity))
    return out[:count]


def bcast_round(q: int, n: int, j: int):
    k = ctypes.c_int32(0)
    shift = ctypes.c_int64(0)
    _check(_load().bcast_round(q, n, j, ctypes.byref(k), ctypes.byref(shift)))
    return int(k.value), int(shift.value)


def bcast_round_block(q: int, n: int, j: int, sched_row) -> int:
    row = np.ascontiguousarray(sched_row, dtype=np.int32)
    rc = int(_load().bcast_round_block(q, n, j, row.ctypes.data))
    if rc < BCAST_NONE:
        raise BcastError(rc)
    return rc


# ------------------------------------------------------------------ device entry points
def bcast_schedule(p: int, root: int, rank_begin: int, rank_end: int, recvblock, sendblock, stream=None) -> int:
    """Fill int32 device tensors [rank_end-rank_begin, q]; either may be None. Returns q."""
    return _check(_load().bcast_schedule(p, root, rank_begin, rank_end, _ptr(recvblock), _ptr(sendblock),
                                         _stream(stream)))


def bcast_schedule_shifted(p: int, root: int, n: int, rank_begin: int, rank_end: int, recvblock, sendblock,
                           stream=None) -> int:
    """bcast_schedule with Algorithm 1's preamble for n blocks applied to every row. Returns q."""
    return _check(_load().bcast_schedule_shifted(p, root, n, rank_begin, rank_end, _ptr(recvblock),
                                                 _ptr(sendblock), _stream(stream)))


def bcast_simulate_scratch_bytes(p: int, n: int, reduction: bool = False) -> int:
    return _check(_load().bcast_simulate_scratch_bytes(p, n, 1 if reduction else 0))


def bcast_simulate_broadcast(p: int, root: int, n: int, recvblock, sendblock, arrival, stats, scratch,
                             stream=None) -> int:
    """Algorithm 1 by all processors on device tables [p, q]: fills arrival [n, p] int32 and stats [8] uint64."""
    nbytes = 0 if scratch is None else scratch.numel() * scratch.element_size()
    return _check(_load().bcast_simulate_broadcast(p, root, n, _ptr(recvblock), _ptr(sendblock), _ptr(arrival),
                                                   _ptr(stats), _ptr(scratch), nbytes, _stream(stream)))


def bcast_simulate_reduce(p: int, root: int, n: int, recvblock, sendblock, value, result, stats, scratch,
                          stream=None) -> int:
    """The reversed rounds as a wrapping-sum reduction of value [n, p] (uint64 bits); result [n], stats [8]."""
    nbytes = 0 if scratch is None else scratch.numel() * scratch.element_size()
    return _check(_load().bcast_simulate_reduce(p, root, n, _ptr(recvblock), _ptr(sendblock), _ptr(value),
                                                _ptr(result), _ptr(stats), _ptr(scratch), nbytes, _stream(stream)))


def bcast_simulate_all_scratch_bytes(p: int, n: int, reduction: bool = False) -> int:
    return _check(_load().bcast_simulate_all_scratch_bytes(p, n, 1 if reduction else 0))


def bcast_simulate_allbroadcast(p: int, n: int, recvblock, sendblock, arrival, stats, scratch, stream=None) -> int:
    nbytes = scratch.numel() * scratch.element_size() if scratch is not None else 0
    return _check(_load().bcast_simulate_allbroadcast(p, n, _ptr(recvblock), _ptr(sendblock), _ptr(arrival),
                                                      _ptr(stats), _ptr(scratch), nbytes, _stream(stream)))


def bcast_simulate_allreduce(p: int, n: int, recvblock, sendblock, value, result, stats, scratch,
                             stream=None) -> int:
    nbytes = scratch.numel() * scratch.element_size() if scratch is not None else 0
    return _check(_load().bcast_simulate_allreduce(p, n, _ptr(recvblock), _ptr(sendblock), _ptr(value),
                                                   _ptr(result), _ptr(stats), _ptr(scratch), nbytes,
                                                   _stream(stream)))


def bcast_allbroadcast_schedule(p: int, rank: int, root_begin: int, root_end: int, recvblocks, sendblocks,
                                stream=None) -> int:
    """Algorithm 7's tables of processor `rank`: row j-root_begin is its schedule with j as root. Returns q."""
    return _check(_load().bcast_allbroadcast_schedule(p, rank, root_begin, root_end, _ptr(recvblocks),
                                                      _ptr(sendblocks), _stream(stream)))


def bcast_schedule_host(p: int, root: int, rank_begin: int, rank_end: int, recvblock_host, sendblock_host,
                        staging, stream=None) -> int:
    """Host (ideally pinned) int32 output tables, filled chunk by chunk through a device staging tensor."""
    nbytes = staging.numel() * staging.element_size()
    return _check(_load().bcast_schedule_host(p, root, rank_begin, rank_end, _ptr(recvblock_host),
                                              _ptr(sendblock_host), _ptr(staging), nbytes, _stream(stream)))


def bcast_schedule_batch(p, rank, root, row_stride: int, recvblock, sendblock, bad_count=None, stream=None) -> int:
    nq = p.numel()
    return _check(_load().bcast_schedule_batch(_ptr(p), _ptr(rank), _ptr(root), nq, row_stride,
                                               _ptr(recvblock), _ptr(sendblock), _ptr(bad_count), _stream(stream)))


def bcast_verify_sweep_scratch_bytes(p_lo: int, p_hi: int) -> int:
    return _check(_load().bcast_verify_sweep_scratch_bytes(p_lo, p_hi))


def bcast_verify_sweep(p_lo: int, p_hi: int, checksum, fail_counts, scratch, stream=None) -> int:
    nbytes = scratch.numel() * scratch.element_size()
    return _check(_load().bcast_verify_sweep(p_lo, p_hi, _ptr(checksum), _ptr(fail_counts), _ptr(scratch),
                                             nbytes, _stream(stream)))


def bcast_verify_sweep_static(p_lo: int, p_hi: int, checksum, fail_counts, stream=None) -> int:
    """The sweep for callers that may not allocate: its tables live in an 8 MiB array inside the library.

    checksum / fail_counts are the caller's device tensors as for bcast_verify_sweep; p_hi <= 65536.
    Calls share the array, so calls that could overlap on the device must be serialised.
    """
    return _check(_load().bcast_verify_sweep_static(p_lo, p_hi, _ptr(checksum), _ptr(fail_counts),
                                                    _stream(stream)))


# ------------------------------------------------------------------ conveniences (allocation only)
def schedule(p: int, root: int = 0, rank_begin: int = 0, rank_end: int | None = None, device="cuda",
             want_recv: bool = True, want_send: bool = True):
    """Allocate and fill (recvblock, sendblock) int32 device tensors for the rank range."""
    import torch
    if rank_end is None:
        rank_end = p
    q = bcast_q(p)
    rows = max(rank_end - rank_begin, 0)
    recv = torch.empty((rows, q), dtype=torch.int32, device=device) if want_recv else None
    send = torch.empty((rows, q), dtype=torch.int32, device=device) if want_send else None
    bcast_schedule(p, root, rank_begin, rank_end, recv, send)
    return recv, send


def allbroadcast_schedule(p: int, rank: int, root_begin: int = 0, root_end: int | None = None, device="cuda"):
    """Allocate and fill Algorithm 7's (recvblocks, sendblocks) of processor `rank` for the roots given."""
    import torch
    if root_end is None:
        root_end = p
    q = bcast_q(p)
    rows = max(root_end - root_begin, 0)
    recv = torch.empty((rows, q), dtype=torch.int32, device=device)
    send = torch.empty((rows, q), dtype=torch.int32, device=device)
    bcast_allbroadcast_schedule(p, rank, root_begin, root_end, recv, send)
    return recv, send


def schedule_batch(p, rank, root, row_stride: int = BCAST_MAX_Q):
    """Allocate and fill padded rows for device int32 query tensors; returns (recv, send, bad_count)."""
    import torch
    nq = p.numel()
    recv = torch.empty((nq, row_stride), dtype=torch.int32, device=p.device)
    send = torch.empty((nq, row_stride), dtype=torch.int32, device=p.device)
    bad = torch.zeros(1, dtype=torch.int32, device=p.device)
    bcast_schedule_batch(p, rank, root, row_stride, recv, send, bad)
    return recv, send, bad


def verify_sweep(p_lo: int, p_hi: int, device="cuda"):
    """Allocate buffers, run the fused verification sweep; returns (checksums uint64 as int64 tensor, fail_counts)."""
    import torch
    checksum = torch.zeros(p_hi - p_lo + 1, dtype=torch.int64, device=device)
    fails = torch.zeros(8, dtype=torch.int32, device=device)
    scratch = torch.empty(bcast_verify_sweep_scratch_bytes(p_lo, p_hi), dtype=torch.uint8, device=device)
    bcast_verify_sweep(p_lo, p_hi, checksum, fails, scratch)
    return checksum, fails


def simulate_broadcast(p: int, root: int, n: int, recvblock, sendblock):
    """Allocate buffers and run Algorithm 1 on the tables; returns (arrival [n, p] int32, stats [8] as int64 bits)."""
    import torch
    dev = recvblock.device if recvblock is not None else "cuda"
    arrival = torch.empty((n, p), dtype=torch.int32, device=dev)
    stats = torch.empty(8, dtype=torch.int64, device=dev)
    scratch = torch.empty(bcast_simulate_scratch_bytes(p, n), dtype=torch.uint8, device=dev)
    bcast_simulate_broadcast(p, root, n, recvblock, sendblock, arrival, stats, scratch)
    return arrival, stats


def simulate_reduce(p: int, root: int, n: int, recvblock, sendblock, value):
    """Allocate buffers and run the reduction on a copy of value [n, p] (int64 tensor holding uint64 bits);
    returns (result [n], stats [8]) as int64 bit patterns."""
    import torch
    work = value.clone()
    result = torch.empty(n, dtype=torch.int64, device=value.device)
    stats = torch.empty(8, dtype=torch.int64, device=value.device)
    scratch = torch.empty(bcast_simulate_scratch_bytes(p, n, True), dtype=torch.uint8, device=value.device)
    bcast_simulate_reduce(p, root, n, recvblock, sendblock, work, result, stats, scratch)
    return result, stats


def simulate_allbroadcast(p: int, n: int, recvblock, sendblock):
    """Allocate state and scratch and run Algorithm 7 by all processors on root-0 tables: (arrival [p][n][p], stats)."""
    import torch
    arrival = torch.empty((p, n, p), dtype=torch.int32, device="cuda")
    stats = torch.zeros(8, dtype=torch.int64, device="cuda")
    scratch = torch.empty(max(bcast_simulate_all_scratch_bytes(p, n), 16), dtype=torch.uint8, device="cuda")
    bcast_simulate_allbroadcast(p, n, recvblock, sendblock, arrival, stats, scratch)
    return arrival, stats


def simulate_allreduce(p: int, n: int, recvblock, sendblock, value):
    """The all-reduction on root-0 tables; value [p][n][p] uint64 (as int64 tensor) is copied.  Returns (result [p][n], stats)."""
    import torch
    work = value.clone()
    result = torch.empty((p, n), dtype=torch.int64, device="cuda")
    stats = torch.zeros(8, dtype=torch.int64, device="cuda")
    scratch = torch.empty(max(bcast_simulate_all_scratch_bytes(p, n, True), 16), dtype=torch.uint8, device="cuda")
    bcast_simulate_allreduce(p, n, recvblock, sendblock, work, result, stats, scratch)
    return result, stats
