"""The decode kernel's CTAs normally hand one another their share of the LoRA shrink result, but
none of them depends on it: after a bounded wait a CTA computes all of it itself, with the same
arithmetic.  The wait (LML_DECODE_PATIENCE, in SM clock cycles) is read once per process; a child
process with patience 0 sends every CTA down the self-sufficient path.  Its outputs must equal the
normal path's bit for bit and agree with the oracle, and the table's counters must be left clean
(a second call in the same process works and gives the same result)."""
import os
import subprocess
import sys

import numpy as np
import pytest

pytestmark = pytest.mark.gpu

ROOT = os.path.dirname(os.path.dirname(os.path.abspath(__file__)))

CHILD = r"""
import sys
sys.path.insert(0, %r); sys.path.insert(0, %r)
import numpy as np
import oracle
from paper_2608_15241_b200 import workloads as wl
from gpu_util import Site
out = {}
cases = [wl.ragged(T=8, d_in=264, d_out=136, ranks=(4, 16, 1, 33, 64)),
         wl.ragged(T=16, d_in=520, d_out=264, ranks=(4, 16, 1, 33, 64)),
         wl.ragged(T=16, d_in=1024, d_out=4104, ranks=(64, 64, 64, 64, 64), shuffled=True),
         wl.ragged(T=5, d_in=4096, d_out=512, ranks=(16, 16, 16, 16, 16)),
         # CTAs with several rounds of rows: the expand of early rounds is put off until u is there
         wl.ragged(T=8, d_in=264, d_out=5200, ranks=(4, 16, 1, 33, 64)),
         wl.ragged(T=16, d_in=264, d_out=10360, ranks=(8, 16, 16, 64, 2), shuffled=True),
         wl.ragged(T=3, d_in=4104, d_out=16000, ranks=(16, 16, 16, 16, 16)),
         # rows of x wider than one pass through the staging buffer: pairs in registers, staged groups of four
         wl.ragged(T=16, d_in=4104, d_out=512, ranks=(16, 16, 16, 16, 16)),
         wl.ragged(T=16, d_in=8200, d_out=264, ranks=(64, 64, 33, 16, 64))]
for i, w in enumerate(cases):
    site = Site(w)
    y, flags = site.run()
    ref, _ = oracle.forward_workload(w)
    r = oracle.compare(y, ref)
    assert flags == 0 and r["ok"], (i, flags, r)
    y2, flags2 = site.run()
    assert flags2 == 0 and np.array_equal(y, y2), i
    out["y%%d" %% i] = y
    site.close()
np.savez(sys.argv[1], **out)
print("decode cases ok")
""" % (ROOT, os.path.join(ROOT, "tests"))


def _run(tmp_path, name, patience):
    env = dict(os.environ)
    env.pop("LML_DECODE_PATIENCE", None)
    if patience is not None:
        env["LML_DECODE_PATIENCE"] = str(patience)
    path = str(tmp_path / name)
    p = subprocess.run([sys.executable, "-c", CHILD, path], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stdout + p.stderr
    assert "decode cases ok" in p.stdout
    return np.load(path)


def test_self_sufficient_path_matches_normal_path(tmp_path):
    normal = _run(tmp_path, "normal.npz", None)
    alone = _run(tmp_path, "alone.npz", 0)
    assert sorted(normal.files) == sorted(alone.files) and len(normal.files) == 9
    for k in normal.files:
        assert np.array_equal(normal[k], alone[k]), k
