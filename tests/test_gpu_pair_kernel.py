"""The CTA-pair (cta_group::2) GEMM kernel is not the default path, so the ordinary parity tests do
not reach it.  The knob LML_FORCE_GEMM=pair is read once per process; this test runs the parity cases
in a child process with the knob set and compares with the oracle there."""
import os
import subprocess
import sys

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
cases = [wl.tiny(), wl.lattice(), wl.ragged(), wl.ragged(shuffled=True),
         wl.ragged(T=129, d_in=200, d_out=264, ranks=(4, 16, 1, 33, 64)),
         wl.ragged(T=333, d_in=1096, d_out=1288, ranks=(8, 16, 32, 64, 4)),
         wl.ragged(T=600, d_in=256, d_out=512)]
for w in cases:
    site = Site(w)
    y, flags = site.run()
    ref, _ = oracle.forward_workload(w)
    r = oracle.compare(y, ref)
    assert flags == 0 and r["ok"], (w.name, w.T, flags, r)
    if w.name == "lattice":
        assert np.array_equal(wl.bf16_bits_to_f64(y), ref)
    y0, flags = site.run(seg_offsets=[0], seg_entry=[])
    base = oracle.forward(w.x, w.W0, [], [0, w.T], [-1])[0]
    assert flags == 0 and oracle.compare(y0, base)["ok"], w.name
    site.close()
print("pair kernel parity ok")
""" % (ROOT, os.path.join(ROOT, "tests"))


def test_pair_kernel_parity_in_child_process():
    env = dict(os.environ, LML_FORCE_GEMM="pair")
    p = subprocess.run([sys.executable, "-c", CHILD], env=env, capture_output=True, text=True, timeout=300)
    assert p.returncode == 0, p.stdout + p.stderr
    assert "pair kernel parity ok" in p.stdout
