"""The LoRA shrink inside the GEMM kernel (whole-K tiles: the CTAs with the fewest output tiles first compute
u = scale * x.A^T for a row tile each on the tensor cores and raise a flag per row tile) against the oracle and
against the separate shrink kernel (LML_FUSE_SHRINK=0, read when a table is created): the two differ only in
the rounding of u to bf16.  Shapes are such that the library chooses the fused form (256-column tiles in more than one wave)."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import Site

pytestmark = pytest.mark.gpu


def _both(w, monkeypatch, **run_kw):
    monkeypatch.delenv("LML_FUSE_SHRINK", raising=False)
    site = Site(w)
    y_fused, f1 = site.run(**run_kw)
    y_again, _ = site.run(**run_kw)
    launches = site.table.last_launch_count()
    site.close()
    monkeypatch.setenv("LML_FUSE_SHRINK", "0")
    site = Site(w)
    y_plain, f2 = site.run(**run_kw)
    launches_plain = site.table.last_launch_count()
    site.close()
    assert f1 == 0 and f2 == 0
    assert np.array_equal(y_fused, y_again)              # run-to-run bits, and the epoch / flags work call after call
    assert launches == launches_plain - 1                # one kernel fewer
    a, b = wl.bf16_bits_to_f64(y_fused), wl.bf16_bits_to_f64(y_plain)
    assert (np.abs(a - b) <= 2.0 ** -6 * np.maximum(1.0, np.abs(b))).all()
    return y_fused


@pytest.mark.parametrize("kw", [dict(T=700, d_in=520, d_out=8192), dict(T=1300, d_in=1032, d_out=4104, shuffled=True),
                                dict(T=2100, d_in=264, d_out=5000)])
def test_fused_shrink_matches_oracle_and_separate_kernel(kw, monkeypatch):
    w = wl.ragged(ranks=(4, 16, 1, 33, 64), **kw)
    y = _both(w, monkeypatch)
    ref, _ = oracle.forward_workload(w)
    r = oracle.compare(y, ref)
    assert r["ok"], r


def test_many_segments_in_one_row_tile_take_several_passes(monkeypatch):
    # 14 segments over 700 rows: several pieces in a 128-row tile, each a pass of its own on another CTA
    w = wl.ragged(T=700, d_in=520, d_out=8192, ranks=(8, 16, 4, 32, 64))
    rng = np.random.default_rng(5)
    cuts = np.sort(rng.integers(0, w.T + 1, size=13))
    so = np.concatenate([[0], cuts, [w.T]]).astype(np.int32)
    se = rng.integers(-1, len(w.entries), size=14).astype(np.int32)
    y = _both(w, monkeypatch, seg_offsets=so, seg_entry=se, perm=None)
    ref, _ = oracle.forward(w.x, w.W0, w.entries, so, se)
    r = oracle.compare(y, ref)
    assert r["ok"], r


def test_malformed_offsets_are_caught_by_the_fused_form(monkeypatch):
    from paper_2608_15241_b200 import binding
    monkeypatch.delenv("LML_FUSE_SHRINK", raising=False)
    w = wl.ragged(T=700, d_in=520, d_out=8192, ranks=(8, 16, 4))
    T = w.T
    site = Site(w)
    y, flags = site.run(seg_offsets=[0, 2 * T // 3, T // 3, T], raw_slot_ids=[site.slots[0], site.slots[1], site.slots[2]])
    assert flags & binding.FLAG_BAD_OFFSETS
    base = oracle.forward(w.x, w.W0, [], [0, T], [-1])[0]
    assert oracle.compare(y, base)["ok"]
    y2, flags2 = site.run(seg_offsets=[0, T // 3, 2 * T // 3, T], raw_slot_ids=[site.slots[0], 7, site.slots[2]])
    assert flags2 & binding.FLAG_BAD_SLOT
    good, f3 = site.run(seg_offsets=[0, T // 3, 2 * T // 3, T], raw_slot_ids=[site.slots[0], -1, site.slots[2]])
    assert f3 == 0 and np.array_equal(y2, good)
    site.close()
