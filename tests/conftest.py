import os
import sys

import pytest

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))
if ROOT not in sys.path:
    sys.path.insert(0, ROOT)

GOLDEN = os.path.join(ROOT, "tests", "golden")


def pytest_configure(config):
    config.addinivalue_line("markers", "gpu: needs a CUDA device (run with -m gpu on a B200)")


def load_golden(name):
    """Parse a golden text fixture: '#' comments, then 'key v0 v1 ...' lines of integers."""
    out = {}
    with open(os.path.join(GOLDEN, name)) as fh:
        for line in fh:
            line = line.strip()
            if not line or line.startswith("#"):
                continue
            toks = line.split()
            out[toks[0]] = [int(t) for t in toks[1:]]
    return out


@pytest.fixture(scope="session")
def golden():
    return load_golden


@pytest.fixture
def forced_shape():
    """forced_shape("block" | "warps" | "lowframe" | "tight" | "auto") forces a launch shape of the table kernel for
    the rest of the test; the per-call choice is restored afterwards."""
    import paper_2407_18004_b200 as bs
    names = {"auto": bs.BCAST_SHAPE_AUTO, "block": bs.BCAST_SHAPE_BLOCK, "warps": bs.BCAST_SHAPE_WARPS,
             "lowframe": bs.BCAST_SHAPE_LOWFRAME, "tight": bs.BCAST_SHAPE_WARPS_TIGHT}
    yield lambda name: bs.bcast_set_launch_shape(names[name])
    bs.bcast_set_launch_shape(bs.BCAST_SHAPE_AUTO)
