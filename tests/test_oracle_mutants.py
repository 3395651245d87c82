"""Do the pins bite?  Each case plants one plausible mistake in a COPY of the oracle's C source
(a dropped term, a wrong comparison, a transposed direction, a missing unlink ...), builds it, and
runs the pin suite against it in a subprocess: the suite must fail.  Nothing here touches the CUDA
path; the mistakes live on the CPU, in the oracle."""
import os
import subprocess
import sys

import pytest

from conftest import ROOT

SOURCE = os.path.join(ROOT, "oracle", "bcast_oracle.c")

MUTANTS = [
    ("skips round down", "skip[k - 1] = skip[k] - skip[k] / 2;", "skip[k - 1] = skip[k] / 2;"),
    ("baseblock never looks at skip[0]", "    } while (k != 0);\n    return c->q;", "    } while (k != 1);\n    return c->q;"),
    ("search: strict first test", "if (rp + skip[e] <= r - skip[k] && rp + skip[e] < s) {",
     "if (rp + skip[e] < r - skip[k] && rp + skip[e] < s) {"),
    ("search: previous position not excluded", "if (rp + skip[e] <= r - skip[k] && rp + skip[e] < s) {",
     "if (rp + skip[e] <= r - skip[k]) {"),
    ("search: recursion one level early", "if (rp + skip[e] <= r - skip[k + 1]) {",
     "if (rp + skip[e] <= r - skip[k]) {"),
    ("search: return test dropped", "if (rp > r - skip[k + 1]) return k;", ";"),
    ("search: accepted index stays in the list", "            NEXT(c, PREV(c, e)) = NEXT(c, e);\n            PREV(c, NEXT(c, e)) = PREV(c, e);\n        }\n        first = 0;",
     "        }\n        first = 0;"),
    ("search: s not kept", "s = rp + skip[e];", ";"),
    ("baseblock stays in the list", "    NEXT(c, PREV(c, b)) = NEXT(c, b);\n    PREV(c, NEXT(c, b)) = PREV(c, b);\n    k = allblocks_",
     "    k = allblocks_"),
    ("search starts at p instead of p + r", "k = allblocks_(c, c->p + r, 0, c->p + c->p, q, 0, 0);",
     "k = allblocks_(c, c->p, 0, c->p + c->p, q, 0, 0);"),
    ("negative blocks off by one", "else recvblock[k] = c->recvblock[k] - q;", "else recvblock[k] = c->recvblock[k] - q + 1;"),
    ("send reads the from-processor", "int64_t t = (a + c.skip[k]) % p;     /* actual to-processor */",
     "int64_t t = (a - c.skip[k] + p) % p;"),
    ("send definition: wrong round", "sendblock[k] = tmp[k];\n    }\n    return c.q;", "sendblock[k] = tmp[k > 0 ? k - 1 : 0];\n    }\n    return c.q;"),
    ("Algorithm 6: bound not lowered", "if (e > c.skip[k]) e = c.skip[k];", ";"),
    ("Algorithm 6: sendblock[0]", "if (q > 0) sendblock[0] = b - q;", "if (q > 0) sendblock[0] = b;"),
    ("round lookup: x", "x = (q - (n - 1) % q) % q;\n    for (i = 0; i < q; i++) {", "x = (n - 1) % q;\n    for (i = 0; i < q; i++) {"),
    ("Algorithm 7: wrong direction of the root offset", "int64_t rp = (r - j + p) % p;", "int64_t rp = (j - r + p) % p;"),
    ("Algorithm 7: send rows from the to-side", "int64_t f = (j - c.skip[k] + p) % p;", "int64_t f = (j + c.skip[k]) % p;"),
    ("root renumbering", "int64_t r = (a - root + p) % p;\n                recvschedule_(&c, r, tmp, NULL);\n                for (k = 0; k < q; k++) recv_tab",
     "int64_t r = (a + root) % p;\n                recvschedule_(&c, r, tmp, NULL);\n                for (k = 0; k < q; k++) recv_tab"),
    ("Algorithm 1's preamble: virtual rounds include x", "if (i < x) tab[a * q + i] += q;", "if (i <= x) tab[a * q + i] += q;"),
    ("simulated broadcast: virtual rounds not moved to the next phase",
     "if (i < x) { rb[a * q + i] += q; sb[a * q + i] += q; }", ";"),
    ("simulated broadcast: rounds counted from the virtual ones", "int64_t round = i - x + 1;", "int64_t round = i + 1;"),
    ("simulated broadcast: sender's holdings not checked", "} else if (!wire_held[f]) {", "} else if (0) {"),
    ("simulated reduction: partial results travel the broadcast's way",
     "int64_t t = (a + skip[k]) % p;\n            int32_t sv", "int64_t t = (a - skip[k] + p) % p;\n            int32_t sv"),
    ("simulated reduction: received value replaces the partial result", "value[want * p + a] += wire_val[t];",
     "value[want * p + a] = wire_val[t];"),
    ("simulated reduction: rounds not reversed", "for (i = n + q - 1 + x - 1; i >= x; i--) {",
     "for (i = x; i < n + q - 1 + x; i++) {"),
    ("all-broadcast: the sender leaves out its own root instead of the to-processor's",
     "if (j != t) blk = round_block_(sends[", "if (j != r) blk = round_block_(sends["),
    ("all-broadcast: unpacked from the to-processor's message",
     "int64_t f = (r - skip[k] + p) % p;\n            for (j = 0; j < p; j++) {\n                int64_t want;",
     "int64_t f = (r + skip[k]) % p;\n            for (j = 0; j < p; j++) {\n                int64_t want;"),
    ("all-broadcast: processor r reads root j's row at (j - r) mod p", "int64_t v = (r - j + p) % p;",
     "int64_t v = (j - r + p) % p;"),
    ("all-broadcast: blocks not shifted by the virtual rounds", "blk = (int64_t)entry + (i / q) * q - x;",
     "blk = (int64_t)entry + (i / q) * q;"),
    ("all-reduction: a partial result expected from a root for its own blocks", "if (j != t) want = round_block_(sends[",
     "if (1) want = round_block_(sends["),
    ("all-reduction: received value replaces the partial result",
     "value[(j * n + want) * p + r] += wire_val[t * p + j];", "value[(j * n + want) * p + r] = wire_val[t * p + j];"),
]


@pytest.mark.parametrize("name,old,new", MUTANTS, ids=[m[0] for m in MUTANTS])
def test_planted_mistake_is_caught(tmp_path, name, old, new):
    source = open(SOURCE).read()
    assert source.count(old) >= 1, "the mutation's anchor is gone from the oracle source"
    mutant_c = tmp_path / "mutant.c"
    mutant_so = tmp_path / "mutant.so"
    mutant_c.write_text(source.replace(old, new, 1))
    subprocess.check_call(["gcc", "-O1", "-std=c99", "-shared", "-fPIC", "-o", str(mutant_so), str(mutant_c)])
    env = dict(os.environ, ORACLE_LIBRARY=str(mutant_so))
    run = subprocess.run([sys.executable, "-m", "pytest", os.path.join(ROOT, "tests", "test_oracle_pins.py"),
                          "-x", "-q", "-p", "no:cacheprovider"], capture_output=True, text=True, env=env, cwd=ROOT,
                         timeout=600)
    # a failing assertion or a crash of the broken build both count; a clean pass does not
    assert run.returncode != 0, f"no pin noticed: {name}"
