"""CPU-side tests of the CUDA library: it loads, exports what the header declares,
its host-only entry points agree with the oracle, and bad arguments are refused
before anything is launched (no GPU needed for any of this)."""
import ctypes
import os
import re

import numpy as np
import pytest

import oracle
import paper_2407_18004_b200 as bs
from conftest import ROOT


def declared_functions():
    text = open(os.path.join(ROOT, "include", "bcast_sched.h")).read()
    text = re.sub(r"/\*.*?\*/", "", text, flags=re.S)
    names = set(re.findall(r"\b(bcast_[a-z_0-9]+)\s*\(", text))
    return sorted(n for n in names if not n.endswith("_inline"))      # inline helpers are not exported


def test_library_exports_every_declared_symbol():
    lib = ctypes.CDLL(bs.library_path())
    names = declared_functions()
    assert {"bcast_q", "bcast_skips", "bcast_schedule", "bcast_schedule_host", "bcast_schedule_batch",
            "bcast_allbroadcast_schedule", "bcast_verify_sweep_static", "bcast_schedule_shifted",
            "bcast_simulate_scratch_bytes", "bcast_simulate_broadcast", "bcast_simulate_reduce",
            "bcast_verify_sweep", "bcast_verify_sweep_scratch_bytes", "bcast_round", "bcast_round_block",
            "bcast_strerror"} <= set(names)
    for name in names:
        assert hasattr(lib, name), name


def test_q_and_skips_match_oracle():
    rng = np.random.default_rng(7)
    ps = list(range(1, 2000)) + [int(x) for x in rng.integers(2000, 2 ** 31 - 1, 2000)] + [2 ** 31 - 1, 2 ** 27 - 1]
    for p in ps:
        assert bs.bcast_q(p) == oracle.q_of(p)
        assert bs.bcast_skips(p).tolist() == oracle.skips(p).tolist()


def test_round_lookup_matches_oracle():
    rng = np.random.default_rng(8)
    for q in range(1, 12):
        for n in list(range(1, 40)) + [1000, 12345]:
            row = rng.integers(-q, q, q).astype(np.int32)
            total = n - 1 + q
            js = range(total) if total < 80 else [0, 1, q, total // 2, total - 2, total - 1]
            for j in js:
                k, shift = bs.bcast_round(q, n, j)
                assert k == oracle.round_k(q, n, j)
                assert bs.bcast_round_block(q, n, j, row) == oracle.round_block(q, n, j, row)
                x = (q - (n - 1) % q) % q
                assert shift == q * ((x + j) // q) - x


def test_inline_round_lookup_compiles_as_c_and_matches_oracle(tmp_path):
    # the header's inline form of the lookup, built with a plain C compiler
    import subprocess
    src = tmp_path / "shim.c"
    src.write_text('#include "bcast_sched.h"\n'
                   'long long shim(int q, long long n, long long j, const int *row, int *k)\n'
                   '{ return bcast_round_block_inline(q, n, j, row, k); }\n')
    lib_path = tmp_path / "shim.so"
    subprocess.check_call(["gcc", "-std=c99", "-Wall", "-Werror", "-shared", "-fPIC", "-I", os.path.join(ROOT, "include"),
                           "-o", str(lib_path), str(src)])
    shim = ctypes.CDLL(str(lib_path)).shim
    shim.restype = ctypes.c_longlong
    shim.argtypes = [ctypes.c_int, ctypes.c_longlong, ctypes.c_longlong, ctypes.c_void_p, ctypes.POINTER(ctypes.c_int)]
    rng = np.random.default_rng(9)
    for q in range(1, 12):
        for n in list(range(1, 30)) + [1000]:
            row = rng.integers(-q, q, q).astype(np.int32)
            total = n - 1 + q
            for j in (range(total) if total < 60 else [0, 1, q, total // 2, total - 1]):
                k = ctypes.c_int(-1)
                assert shim(q, n, j, row.ctypes.data, ctypes.byref(k)) == oracle.round_block(q, n, j, row)
                assert k.value == oracle.round_k(q, n, j)


def test_host_argument_errors():
    assert bs.bcast_strerror(0) == "success"
    for code in range(-10, 0):
        assert bs.bcast_strerror(code) not in ("", "success")
    with pytest.raises(bs.BcastError) as e:
        bs.bcast_q(0)
    assert e.value.code == -1
    with pytest.raises(bs.BcastError) as e:
        bs.bcast_round(0, 3, 0)
    assert e.value.code == -6
    with pytest.raises(bs.BcastError) as e:
        bs.bcast_round(4, 3, 6)
    assert e.value.code == -7
    with pytest.raises(bs.BcastError) as e:
        bs.bcast_round_block(4, 3, -1, [0, 0, 0, 0])
    assert e.value.code == -7
    with pytest.raises(bs.BcastError) as e:
        bs.bcast_set_simulate_rounds(4)
    assert e.value.code == -12
    for mode in (bs.BCAST_ROUNDS_FUSED, bs.BCAST_ROUNDS_LAUNCHES, bs.BCAST_ROUNDS_AUTO):
        assert bs.bcast_set_simulate_rounds(mode) == 0
    lib = ctypes.CDLL(bs.library_path())
    lib.bcast_schedule.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_int64, ctypes.c_int64,
                                   ctypes.c_void_p, ctypes.c_void_p, ctypes.c_void_p]
    fake = ctypes.c_void_p(0x1000)     # never dereferenced: every call below fails its checks first
    assert lib.bcast_schedule(0, 0, 0, 0, fake, fake, None) == -1
    assert lib.bcast_schedule(10, 10, 0, 10, fake, fake, None) == -2
    assert lib.bcast_schedule(10, -1, 0, 10, fake, fake, None) == -2
    assert lib.bcast_schedule(10, 0, 5, 4, fake, fake, None) == -3
    assert lib.bcast_schedule(10, 0, 0, 11, fake, fake, None) == -3
    assert lib.bcast_schedule(10, 0, 0, 10, None, None, None) == -4
    assert lib.bcast_schedule(10, 0, 0, 10, ctypes.c_void_p(0x1002), None, None) == -5
    assert lib.bcast_schedule(1, 0, 0, 1, fake, fake, None) == 0          # q = 0: nothing to launch
    assert lib.bcast_schedule(10, 0, 3, 3, fake, fake, None) == 4         # empty range
    lib.bcast_schedule_batch.argtypes = [ctypes.c_void_p] * 3 + [ctypes.c_int64, ctypes.c_int32] + [ctypes.c_void_p] * 4
    assert lib.bcast_schedule_batch(fake, fake, fake, 5, 30, fake, fake, None, None) == -9
    assert lib.bcast_schedule_batch(fake, fake, fake, -1, 31, fake, fake, None, None) == -6
    assert lib.bcast_schedule_batch(None, fake, fake, 5, 31, fake, fake, None, None) == -4
    assert lib.bcast_schedule_batch(fake, fake, fake, 5, 31, None, None, None, None) == -4
    assert lib.bcast_schedule_batch(fake, fake, fake, 0, 31, fake, fake, None, None) == 0
    lib.bcast_verify_sweep.argtypes = [ctypes.c_int32, ctypes.c_int32, ctypes.c_void_p, ctypes.c_void_p,
                                       ctypes.c_void_p, ctypes.c_int64, ctypes.c_void_p]
    assert lib.bcast_verify_sweep(5, 4, fake, fake, fake, 1 << 20, None) == -3
    assert lib.bcast_verify_sweep(0, 4, fake, fake, fake, 1 << 20, None) == -1
    assert lib.bcast_verify_sweep(2, 4, None, fake, fake, 1 << 20, None) == -4
    assert lib.bcast_verify_sweep(2, 1000, fake, fake, fake, 512, None) == -10


def test_workload_generator_is_seeded_and_in_range():
    from paper_2407_18004_b200 import workloads
    p, rank, root = workloads.query_batch(10000, seed=0)
    p2, rank2, root2 = workloads.query_batch(10000, seed=0)
    assert np.array_equal(p, p2) and np.array_equal(rank, rank2) and np.array_equal(root, root2)
    assert p.min() >= 2 and (rank >= 0).all() and (rank < p).all() and (root >= 0).all() and (root < p).all()
    # log-uniform: every octave between 2^1 and 2^31 is populated
    octave = np.floor(np.log2(p.astype(np.float64))).astype(int)
    assert set(range(1, 31)) <= set(octave.tolist())


def test_low_state_table_matches_oracle_receive_schedules():
    """The table of the search's low states, which the host fills and the table kernel looks undecided low rounds
    up in: every state's rounds against the oracle's receive schedule (Algorithm 5) of ranks in that state."""
    levels = 9
    rng = np.random.default_rng(11)
    ps = [2 ** 11 + 1, 3000, 2 ** 12 - 1, 40001, 2 ** 16 + 1, 2 ** 20 + 1, 3858024, 2 ** 24 + 3, 123456789,
          2 ** 27 - 1, 2 ** 31 - 1]
    assert len(bs.bcast_low_states(1000)) == 0 and len(bs.bcast_low_states(1024)) == 0      # q = 10: not used
    for p in ps:
        q = oracle.q_of(p)
        skip = [int(x) for x in oracle.skips(p)]
        states = bs.bcast_low_states(p)
        assert len(states) == skip[levels] and states[0] == states[1] == 0xFFFFFFFF
        assert list(bs.bcast_low_states(p, 100)) == list(states[:100])
        ranks = range(1, p) if p <= 5000 else [int(x) for x in rng.integers(1, p, 1500)]
        seen = set()
        for r in ranks:
            # what is left of p + r after its greedy digits at the levels >= 9 (skip[q] = p comes first, leaving r)
            u, j = r, q
            for k in range(q - 1, levels - 1, -1):
                if u >= skip[k]:
                    u -= skip[k]
                    j = k
            if u < 2:
                continue
            seen.add(u)
            recv = oracle.recvschedule(p, r)
            popped = oracle.baseblock(p, r) if j == q else j - q
            word = int(states[u])
            rounds = 0
            for k in range(8):
                nib = (word >> (4 * k)) & 15
                if nib == 15:
                    break
                assert int(recv[k]) == (popped if nib == 14 else nib - q), (p, r, u, k, hex(word))
                rounds += 1
                if nib == 14:
                    assert all((word >> (4 * kk)) & 15 == 15 for kk in range(k + 1, 8)), (p, u, hex(word))
                    break
            else:
                assert int(recv[8]) == popped, (p, r, u, hex(word))        # eight rounds used up every low index
            assert rounds >= 1, (p, r, u, hex(word))
        assert len(seen) >= min(200, skip[levels] - 2) or p > 5000, (p, len(seen))


def test_low_state_table_argument_errors():
    buf = np.zeros(8, dtype=np.uint32)
    lib = ctypes.CDLL(bs.library_path())
    lib.bcast_low_states.argtypes = [ctypes.c_int32, ctypes.c_void_p, ctypes.c_int32]
    assert lib.bcast_low_states(0, buf.ctypes.data, 8) == -1
    assert lib.bcast_low_states(5000, None, 8) < 0
    assert lib.bcast_low_states(5000, buf.ctypes.data, -1) < 0
    assert lib.bcast_low_states(5000, buf.ctypes.data, 8) == 8
    assert lib.bcast_low_states(5000, buf.ctypes.data, 0) == 0
