"""The split-K kernel for few tokens (a cluster of CTAs shares one tile, partial sums exchanged through
distributed shared memory): every cluster shape against the oracle, on shapes with ragged edges in
every dimension, with a row permutation, with segments of every rank and without adapters; two calls
give the same bits; and the shape the library picks by itself for few tokens agrees as well."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import Site

pytestmark = pytest.mark.gpu

SHAPES = ["128x2", "128x3", "128x4", "256x2", "256x3", "256x4", "256x5", "256x6", "256x8"]


@pytest.mark.parametrize("shape", SHAPES)
@pytest.mark.parametrize("kw", [dict(T=200, d_in=1032, d_out=520), dict(T=77, d_in=1024, d_out=264, shuffled=True),
                                dict(T=130, d_in=2048, d_out=1000)])
def test_split_shapes_against_oracle(shape, kw, monkeypatch):
    monkeypatch.setenv("LML_GEMM_SPLIT", shape)
    w = wl.ragged(ranks=(4, 16, 1, 33, 64), **kw)
    site = Site(w)
    y, flags = site.run()
    assert flags == 0
    ref, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, w.seg_entry, w.perm)
    r = oracle.compare(y, ref)
    assert r["ok"], (shape, r)
    y2, _ = site.run()
    assert np.array_equal(y, y2)
    # no adapters at all: the base product alone
    yb, fb = site.run(seg_offsets=[0, w.T], raw_slot_ids=[-1])
    refb, _ = oracle.forward(w.x, w.W0, w.entries, np.array([0, w.T], np.int32), np.array([-1], np.int32), w.perm)
    assert fb == 0 and oracle.compare(yb, refb)["ok"]
    site.close()


@pytest.mark.parametrize("T", [17, 64, 128, 129, 300])
def test_library_choice_for_few_tokens(T, monkeypatch):
    monkeypatch.delenv("LML_GEMM_SPLIT", raising=False)
    w = wl.ragged(T=T, d_in=2048, d_out=1544, ranks=(8, 16, 16, 64))
    site = Site(w)
    y, flags = site.run()
    assert flags == 0
    ref, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, w.seg_entry, w.perm)
    assert oracle.compare(y, ref)["ok"]
    site.close()
