"""The allocation-free sweep entry point against the ordinary one.

`bcast_verify_sweep_static` is for callers that are not allowed to allocate device
memory when they need a sweep (inside an allocation-free section, or as a plug-in
that is only handed output buffers); it keeps its working tables in a fixed array
inside the library.  Its checksums and failure counters must be exactly those of
`bcast_verify_sweep` (integer results: equality, no tolerance), also on a second
call, which finds the array as the first call left it.  Collected last on purpose.
"""
import numpy as np
import pytest

import paper_2407_18004_b200 as bs

torch = pytest.importorskip("torch")
pytestmark = pytest.mark.gpu


def test_static_sweep_matches_sweep_twice():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    lo, hi = 2, 3000
    want_sum, want_fail = bs.verify_sweep(lo, hi)          # existing entry point, caller-allocated scratch
    torch.cuda.synchronize()
    assert want_fail.tolist() == [0] * 8
    # outputs are allocated up front; the two calls under test get no new memory
    sums = [torch.zeros(hi - lo + 1, dtype=torch.int64, device="cuda") for _ in range(2)]
    fails = [torch.zeros(8, dtype=torch.int32, device="cuda") for _ in range(2)]
    # a different range in between leaves other contents behind in the shared array
    other_sum = torch.zeros(500, dtype=torch.int64, device="cuda")
    other_fail = torch.zeros(8, dtype=torch.int32, device="cuda")
    bs.bcast_verify_sweep_static(lo, hi, sums[0], fails[0])
    bs.bcast_verify_sweep_static(40001, 40500, other_sum, other_fail)
    bs.bcast_verify_sweep_static(lo, hi, sums[1], fails[1])
    torch.cuda.synchronize()
    for i in range(2):
        assert fails[i].tolist() == want_fail.tolist()
        assert np.array_equal(sums[i].cpu().numpy(), want_sum.cpu().numpy()), f"call {i + 1}"
    ref_sum, ref_fail = bs.verify_sweep(40001, 40500)
    torch.cuda.synchronize()
    assert other_fail.tolist() == [0] * 8 and np.array_equal(other_sum.cpu().numpy(), ref_sum.cpu().numpy())


def test_static_sweep_rejects_oversize():
    if not torch.cuda.is_available():
        pytest.skip("no CUDA device")
    out = torch.zeros(4, dtype=torch.int64, device="cuda")
    fail = torch.zeros(8, dtype=torch.int32, device="cuda")
    with pytest.raises(bs.BcastError) as err:
        bs.bcast_verify_sweep_static(65536, 65537, out, fail)
    assert err.value.code == -11
    with pytest.raises(bs.BcastError):
        bs.bcast_verify_sweep_static(5, 4, out, fail)
