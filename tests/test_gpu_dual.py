"""lora_mixed_linear_dual: the same tokens under two slot bindings, the base product shared.  The first
output must equal the single call with the first binding bit for bit; the second must agree with the
oracle under the second binding (it is the first accumulator plus the difference of the deltas, so it
matches the single call only to fp32 rounding).  Covers segments where a side has no adapter, where
both sides name the same slot, shuffled rows (perm), ragged tails, CTAs with one, two and three
tiles, and the decode form."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import Site, to_bits

pytestmark = pytest.mark.gpu


def _dual(site, w, se_a, se_b):
    import torch
    so = torch.from_numpy(w.seg_offsets).cuda()
    ids_a = torch.from_numpy(site.slot_ids(se_a)).cuda()
    ids_b = torch.from_numpy(site.slot_ids(se_b)).cuda()
    pm = None if w.perm is None else torch.from_numpy(w.perm).cuda()
    y_a, y_b = site.table.lora_mixed_linear_dual(site.x, site.W0, so, ids_a, ids_b, perm=pm)
    torch.cuda.synchronize()
    return to_bits(y_a), to_bits(y_b), site.table.device_status()


@pytest.mark.parametrize("kw", [dict(T=333, d_in=264, d_out=520), dict(T=600, d_in=256, d_out=512, shuffled=True),
                                dict(T=129, d_in=200, d_out=264), dict(T=2100, d_in=512, d_out=5000),
                                dict(T=12, d_in=520, d_out=264), dict(T=300, d_in=40, d_out=136)])
def test_dual_matches_two_single_calls(kw, monkeypatch):
    # (the dual call always runs on whole-K tiles; make the single calls do the same, so that the first
    # output can be compared bit for bit: the split-K kernel for few tokens adds in another order)
    monkeypatch.setenv("LML_GEMM_SPLIT", "0")
    # (and the dual call takes its u blocks from the shrink kernel, while the single call computes them inside the
    # GEMM kernel on the tensor cores: same values to bf16 rounding, not the same bits)
    monkeypatch.setenv("LML_FUSE_SHRINK", "0")
    w = wl.ragged(ranks=(4, 16, 1, 33, 64), **kw)
    E = len(w.entries)
    se_a = w.seg_entry.copy()
    rng = np.random.default_rng(w.T)
    se_b = se_a.copy()
    for g in range(w.G):                       # a different entry, the same one, or none, at random
        se_b[g] = [int(rng.integers(0, E)), se_a[g], -1][int(rng.integers(0, 3))]
    if w.G > 1:
        se_a[0] = -1                           # first binding without an adapter on one segment
    site = Site(w)
    y_a, y_b, flags = _dual(site, w, se_a, se_b)
    assert flags == 0
    y_a1, f1 = site.run(seg_entry=se_a)
    y_b1, f2 = site.run(seg_entry=se_b)
    assert f1 == 0 and f2 == 0
    assert np.array_equal(y_a, y_a1)
    ref_b, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, se_b, w.perm)
    r = oracle.compare(y_b, ref_b)
    assert r["ok"], r
    # against the single call: equal up to the last place of bf16 on almost every element
    diff = np.abs(wl.bf16_bits_to_f64(y_b) - wl.bf16_bits_to_f64(y_b1))
    scale = np.maximum(1.0, np.abs(wl.bf16_bits_to_f64(y_b1)))
    assert (diff <= 2.0 ** -7 * scale).all()
    # a second call on the same table gives the same bits
    y_a2, y_b2, _ = _dual(site, w, se_a, se_b)
    assert np.array_equal(y_a, y_a2) and np.array_equal(y_b, y_b2)
    site.close()


@pytest.mark.parametrize("kw", [dict(T=1, d_in=1032, d_out=2056), dict(T=8, d_in=4096, d_out=4096),
                                dict(T=16, d_in=2056, d_out=1000, shuffled=True), dict(T=11, d_in=264, d_out=40)])
def test_dual_decode_is_one_launch_and_bit_identical_to_two_calls(kw):
    """Up to 16 tokens: one launch of the decode kernel, half of its CTAs per binding, each half a single call."""
    w = wl.ragged(ranks=(4, 16, 1, 33, 64), **kw)
    E = len(w.entries)
    rng = np.random.default_rng(7 + w.T)
    se_a = w.seg_entry.copy()
    se_b = np.array([[int(rng.integers(0, E)), int(se_a[g]), -1][int(rng.integers(0, 3))] for g in range(w.G)], se_a.dtype)
    site = Site(w)
    y_a, y_b, flags = _dual(site, w, se_a, se_b)
    assert flags == 0 and site.table.last_launch_count() == 1
    y_a1, f1 = site.run(seg_entry=se_a)
    y_b1, f2 = site.run(seg_entry=se_b)
    assert f1 == 0 and f2 == 0
    assert np.array_equal(y_a, y_a1) and np.array_equal(y_b, y_b1)
    for y, se in ((y_a, se_a), (y_b, se_b)):
        ref, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, se, w.perm)
        r = oracle.compare(y, ref)
        assert r["ok"], r
    site.close()


@pytest.mark.parametrize("kw", [dict(T=128, d_in=2048, d_out=1544), dict(T=77, d_in=1024, d_out=2056, shuffled=True),
                                dict(T=300, d_in=2048, d_out=1032), dict(T=64, d_in=4096, d_out=4096)])
def test_dual_with_few_tokens_takes_the_split_k_kernel(kw, monkeypatch):
    """The chunk sizes of the paper's stale-coverage prefill (64 to 128 tokens, Section 5.3 / 7.5): the library picks
    the split-K kernel, which multiplies the k-blocks into both bindings' accumulators.  First output bit for bit
    the single call's (same kernel, same order), second within tolerance of the oracle."""
    monkeypatch.delenv("LML_GEMM_SPLIT", raising=False)
    w = wl.ragged(ranks=(4, 16, 1, 33, 64), **kw)
    E = len(w.entries)
    rng = np.random.default_rng(w.T + 1)
    se_a = w.seg_entry.copy()
    se_b = np.array([[int(rng.integers(0, E)), int(se_a[g]), -1][int(rng.integers(0, 3))] for g in range(w.G)], np.int32)
    site = Site(w)
    y_a, y_b, flags = _dual(site, w, se_a, se_b)
    assert flags == 0
    y_a1, f1 = site.run(seg_entry=se_a)
    assert f1 == 0 and np.array_equal(y_a, y_a1)
    for se, y in ((se_a, y_a), (se_b, y_b)):
        ref, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, se, w.perm)
        r = oracle.compare(y, ref)
        assert r["ok"], r
    y_a2, y_b2, _ = _dual(site, w, se_a, se_b)
    assert np.array_equal(y_a, y_a2) and np.array_equal(y_b, y_b2)
    site.close()


def test_dual_on_prefill_q_proj_sampled_rows():
    w = wl.prefill_q_proj()
    se_b = np.roll(w.seg_entry, 1)
    site = Site(w)
    y_a, y_b, flags = _dual(site, w, w.seg_entry, se_b)
    assert flags == 0
    from gpu_util import sample_positions
    pos = sample_positions(w, 48, seed=3)
    for se, y in ((w.seg_entry, y_a), (se_b, y_b)):
        ref, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, se, w.perm, positions=pos)
        rows = pos if w.perm is None else w.perm[pos]
        r = oracle.compare(y[rows], ref[rows])
        assert r["ok"], r
    site.close()
