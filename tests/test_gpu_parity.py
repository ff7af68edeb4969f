"""GPU parity: the CUDA path, called through the C ABI, against the fp64 CPU oracle on the same
seeded inputs.  Criterion (per element and Frobenius) is oracle.compare:
|gpu - oracle| <= 1e-2 * max(1, |oracle|) and ||gpu - oracle||_F / ||oracle||_F <= 5e-3."""
import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

from gpu_util import Site, sample_positions, sample_positions_every_tile, to_bits, to_dev

pytestmark = pytest.mark.gpu


def check_full(w, **site_kw):
    site = Site(w, **site_kw)
    try:
        y, flags = site.run()
        ref, oflags = oracle.forward_workload(w)
        assert flags == 0 and oflags == 0
        r = oracle.compare(y, ref)
        assert r["ok"], r
        return y, ref, r
    finally:
        site.close()


def check_every_tile(w, count=512):
    """Largest shapes: the oracle on >= `count` rows that include a row of every 128-row tile and every
    segment's first and last row (rows are independent, so a sampled row is checked exactly)."""
    site = Site(w)
    try:
        y, flags = site.run()
        assert flags == 0
        pos = sample_positions_every_tile(w, count)
        assert len(pos) >= min(count, w.T)
        ref, _ = oracle.forward_workload(w, positions=pos)
        rows = pos if w.perm is None else w.perm[pos]
        r = oracle.compare(y, ref, rows=rows)
        assert r["ok"], r
        return y
    finally:
        site.close()


# ---- small cases, every element -----------------------------------------------------------------

@pytest.mark.parametrize("kw", [{}, {"zero_base": True}, {"scale_numerator": 100.0},
                                {"zero_base": True, "scale_numerator": 100.0}])
def test_tiny(kw):
    y, ref, r = check_full(wl.tiny(**kw))
    if kw.get("zero_base"):
        # pure LoRA term: a dropped or mis-scaled adapter cannot hide behind the base term
        assert r["rel_fro"] <= 5e-3 and np.abs(ref).max() > 0


def test_lattice_is_exact():
    w = wl.lattice()
    site = Site(w)
    try:
        y, flags = site.run()
        ref, _ = oracle.forward_workload(w)
        assert flags == 0
        assert np.array_equal(wl.bf16_bits_to_f64(y), ref)   # integers: zero error allowed
    finally:
        site.close()


def test_lattice_decode_sizes_are_exact():
    for T in (1, 5, 8, 9, 16):
        w = wl.lattice(T=T, d_in=264, d_out=136)
        w.seg_offsets = np.array([0, T // 2, T], np.int32)
        w.seg_entry = np.array([1, 3], np.int32)
        site = Site(w)
        try:
            y, flags = site.run()
            ref, _ = oracle.forward_workload(w)
            assert flags == 0 and np.array_equal(wl.bf16_bits_to_f64(y), ref), T
        finally:
            site.close()


@pytest.mark.parametrize("shuffled", [False, True])
def test_ragged(shuffled):
    check_full(wl.ragged(shuffled=shuffled))


@pytest.mark.parametrize("T", [17, 127, 128, 129, 300])
def test_ragged_row_counts_around_a_tile(T):
    check_full(wl.ragged(T=T, d_in=200, d_out=264, ranks=(4, 16, 1, 33, 64)))


def test_wide_and_deep_shapes_span_several_tiles():
    # several N tiles with a ragged last one, K not a multiple of 64, 3 row tiles
    check_full(wl.ragged(T=333, d_in=1096, d_out=1288, ranks=(8, 16, 32, 64, 4)))


@pytest.mark.parametrize("T", [1, 2, 7, 8, 9, 15, 16])
def test_decode_token_counts(T):
    w = wl.ragged(T=T, d_in=520, d_out=264, ranks=(4, 16, 1, 33, 64), shuffled=(T % 2 == 1))
    check_full(w)


def test_perm_that_is_the_identity_on_some_tiles():
    # rows 0..255 already in place (two whole tiles are not copied), the rest shuffled
    w = wl.ragged(T=400, d_in=264, d_out=328, ranks=(4, 16, 1, 33, 64))
    rng = np.random.default_rng(5)
    perm = np.arange(w.T, dtype=np.int32)
    perm[256:] = 256 + rng.permutation(w.T - 256)
    w.perm = perm
    site = Site(w)
    try:
        y, flags = site.run()
        ref, _ = oracle.forward_workload(w)
        assert flags == 0 and oracle.compare(y, ref)["ok"]
        # an all-identity perm must give bit for bit what the call without perm gives
        y_id, _ = site.run(perm=np.arange(w.T, dtype=np.int32))
        y_none, _ = site.run(perm=None)
        assert np.array_equal(y_id, y_none)
    finally:
        site.close()


def test_no_segments_means_base_only():
    for T in (8, 200):
        w = wl.ragged(T=T, d_in=136, d_out=200)
        site = Site(w)
        try:
            y, flags = site.run(seg_offsets=[0], seg_entry=[])
            ref, _ = oracle.forward(w.x, w.W0, [], [0, T], [-1])
            assert flags == 0 and oracle.compare(y, ref)["ok"]
        finally:
            site.close()


def test_zero_tokens():
    import torch
    w = wl.tiny()
    site = Site(w)
    try:
        x0 = site.x[:0]
        y = site.table.lora_mixed_linear(x0, site.W0, None, None)
        assert tuple(y.shape) == (0, w.d_out) and site.table.last_launch_count() == 0
    finally:
        site.close()


# ---- the BASELINE configurations ---------------------------------------------------------------------

@pytest.mark.parametrize("split", [False, True])
def test_decode_q_proj(split):
    w = wl.decode_q_proj(split_versions=split)
    y, ref, r = check_full(w)
    # the resident but unbound new version must not have leaked into agent 0's rows
    if not split:
        other = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, np.array([4, 1, 2, 3], np.int32))[0]
        assert not oracle.compare(y, other, rows=np.array([0, 1]))["ok"]


def test_prefill_q_proj_every_element():
    check_full(wl.prefill_q_proj())


def test_prefill_q_proj_shuffled_every_element():
    # the same batch with its rows in arrival order: per-token ids through the segmentation pass, row gather,
    # scatter epilogue
    import torch
    w = wl.shuffle_rows(wl.prefill_q_proj())
    site = Site(w)
    try:
        tok = np.array([site.slots[e] if e >= 0 else -1 for e in w.token_entry], np.int32)
        y = site.table.lora_mixed_linear_tokens(site.x, site.W0, torch.from_numpy(tok).cuda())
        torch.cuda.synchronize()
        assert site.table.device_status() == 0
        ref, _ = oracle.forward_workload(w)
        r = oracle.compare(to_bits(y), ref)
        assert r["ok"], r
    finally:
        site.close()


def test_mlp_up_gate_every_element():
    check_full(wl.mlp_up_gate())


def test_mlp_up_gate_shuffled_through_segmentation_pass_every_element():
    import torch
    w = wl.mlp_up_gate(shuffled=True)
    site = Site(w, max_slots=8)
    try:
        tok = np.array([site.slots[e] if e >= 0 else -1 for e in w.token_entry], np.int32)
        perm, so, ids = site.table.segment_tokens(torch.from_numpy(tok).cuda())
        y = site.table.lora_mixed_linear(site.x, site.W0, so, ids, perm)
        torch.cuda.synchronize()
        assert site.table.device_status() == 0
        assert np.array_equal(perm.cpu().numpy(), w.perm)      # same stable grouping as the recipe
        ref, _ = oracle.forward_workload(w)
        r = oracle.compare(to_bits(y), ref)
        assert r["ok"], r
    finally:
        site.close()


# every cell of the decoder-layer sweep up to 1024 tokens, every element (q k v o share a shape, gate and up too:
# one of each, plus two of the others for their different seeds)
@pytest.mark.parametrize("proj,T", [(p, T) for p in ("q", "gate", "down") for T in (1, 16, 128, 1024)] +
                         [("k", 128), ("up", 1), ("o", 16), ("v", 1024)])
def test_layer_sweep_cells_every_element(proj, T):
    check_full(wl.layer_sweep(proj, T))


# a few blocks of 16 tokens through the token form of the call (one launch of the decode kernel, a share of its CTAs per
# block): every element against the oracle, output and workspace between canary bands
@pytest.mark.parametrize("proj,T", [("q", 17), ("q", 32), ("q", 48), ("down", 31)])
def test_layer_sweep_shapes_at_a_few_blocks_of_tokens(proj, T):
    import torch
    from gpu_util import Guarded
    w = wl.layer_sweep(proj, T)
    site = Site(w)
    try:
        token_entry = np.repeat(w.seg_entry, np.diff(w.seg_offsets))
        if w.perm is not None:
            unperm = np.empty_like(token_entry)
            unperm[w.perm] = token_entry
            token_entry = unperm
        slots = site.slot_ids(token_entry)
        gy = Guarded(T * w.d_out * 2)
        from paper_2608_15241_b200.binding import lml_tokens_workspace_bytes
        gws = Guarded(max(lml_tokens_workspace_bytes(site.table.handle, T), 256))
        y = gy.view(torch.bfloat16, (T, w.d_out))
        site.table.lora_mixed_linear_tokens(site.x, site.W0, torch.from_numpy(slots).cuda(), y=y, workspace=gws.payload)
        torch.cuda.synchronize()
        assert gy.intact() and gws.intact()
        assert site.table.device_status() == 0 and site.table.last_launch_count() == 1
        ref, oflags = oracle.forward_workload(w)
        r = oracle.compare(to_bits(y), ref)
        assert oflags == 0 and r["ok"], r
    finally:
        site.close()


# up to one row tile through the token form of the call beyond the blocks' range: the tokens stay in their order, one
# launch binds them and writes the shrink result slot by slot, the GEMM follows (two launches): every element against
# the oracle, output and workspace between canary bands
@pytest.mark.parametrize("proj,T", [("q", 49), ("q", 64), ("q", 128), ("q", 129), ("q", 256), ("gate", 17), ("gate", 32), ("gate", 128), ("gate", 200), ("down", 33), ("down", 127)])
def test_layer_sweep_shapes_in_one_row_tile_through_the_token_form(proj, T):
    import torch
    from gpu_util import Guarded
    w = wl.layer_sweep(proj, T)
    site = Site(w)
    try:
        token_entry = np.repeat(w.seg_entry, np.diff(w.seg_offsets))
        if w.perm is not None:
            unperm = np.empty_like(token_entry)
            unperm[w.perm] = token_entry
            token_entry = unperm
        slots = site.slot_ids(token_entry)
        gy = Guarded(T * w.d_out * 2)
        from paper_2608_15241_b200.binding import lml_tokens_workspace_bytes
        gws = Guarded(max(lml_tokens_workspace_bytes(site.table.handle, T), 256))
        y = gy.view(torch.bfloat16, (T, w.d_out))
        site.table.lora_mixed_linear_tokens(site.x, site.W0, torch.from_numpy(slots).cuda(), y=y, workspace=gws.payload)
        torch.cuda.synchronize()
        assert gy.intact() and gws.intact()
        assert site.table.device_status() == 0 and site.table.last_launch_count() == 2
        ref, oflags = oracle.forward_workload(w)
        r = oracle.compare(to_bits(y), ref)
        assert oflags == 0 and r["ok"], r
    finally:
        site.close()


# the 8192-token cells: >= 512 rows with a row of every 128-row tile and every segment's ends
@pytest.mark.parametrize("proj", ["o", "gate", "down"])
def test_layer_sweep_8192_token_cells_every_tile(proj):
    check_every_tile(wl.layer_sweep(proj, 8192), count=512)


# ---- properties that hold at any size ----------------------------------------------------------------------

def test_run_to_run_bitwise_determinism_and_unbound_version_changes_nothing():
    w = wl.prefill_q_proj()
    site = Site(w)
    try:
        y1, _ = site.run()
        y2, _ = site.run()
        assert np.array_equal(y1, y2)
        site.table.retire_version(0, 1)          # the resident, unbound old version goes away
        y3, flags = site.run()
        assert flags == 0 and np.array_equal(y1, y3)
    finally:
        site.close()


def test_version_routing_in_one_call():
    # two versions of adapter 0 with B_new = -B_old: rows on old and new differ by twice the delta
    w = wl.ragged(T=260, d_in=256, d_out=320, ranks=(16, 16))
    e0 = w.entries[0]
    w.entries[1] = wl.AdapterEntry(e0.adapter_id, e0.version + 1, e0.rank, e0.scale, e0.A,
                                   (e0.B ^ np.uint16(0x8000)).astype(np.uint16))
    w.seg_offsets = np.array([0, 130, 260], np.int32)
    w.seg_entry = np.array([0, 1], np.int32)
    site = Site(w)
    try:
        y, _ = site.run()
        ref, _ = oracle.forward_workload(w)
        assert oracle.compare(y, ref)["ok"]
        y_swapped, _ = site.run(seg_entry=[1, 0])
        base, _ = oracle.forward(w.x, w.W0, [], [0, w.T], [-1])
        d = wl.bf16_bits_to_f64(y) - base
        ds = wl.bf16_bits_to_f64(y_swapped) - base
        assert np.abs(d + ds).max() <= 2e-2 * max(1.0, np.abs(base).max())
        assert np.abs(d).max() > 0.05
    finally:
        site.close()


def test_adapter_scoped_effect_and_slot_reuse():
    # retiring / re-registering one adapter leaves rows on other adapters bit-identical
    w = wl.ragged(T=300, d_in=256, d_out=320, ranks=(8, 16, 4))
    w.seg_offsets = np.array([0, 100, 200, 300], np.int32)
    w.seg_entry = np.array([0, 1, 2], np.int32)
    site = Site(w, max_slots=3)
    try:
        y1, _ = site.run()
        site.table.retire_version(w.entries[1].adapter_id, w.entries[1].version)
        newA = wl.normal_bf16(9, 1, (32, w.d_in), 0.02)
        newB = wl.normal_bf16(9, 2, (w.d_out, 32), 0.02)
        slot = site.table.register_adapter(77, 5, to_dev(newA), to_dev(newB), 1.0)
        assert slot == site.slots[1]                       # lowest free index is reused
        site.slots[1] = slot
        w.entries[1] = wl.AdapterEntry(77, 5, 32, 1.0, newA, newB)
        y2, flags = site.run()
        assert flags == 0
        assert np.array_equal(y1[:100], y2[:100]) and np.array_equal(y1[200:], y2[200:])
        ref, _ = oracle.forward_workload(w)
        assert oracle.compare(y2, ref)["ok"]
    finally:
        site.close()


def test_segmentation_matches_reference_grouping():
    import torch
    from paper_2608_15241_b200.binding import Table
    tbl = Table(64, 64, max_slots=18)
    try:
        A = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
        B = torch.zeros((64, 4), dtype=torch.bfloat16, device="cuda")
        for a in range(18):
            tbl.register_adapter(a, 1, A, B, 1.0)
        rng = np.random.default_rng(1)
        for T in (0, 1, 31, 32, 33, 1000, 8192, 16384, 16385, 50000):   # (up to 16384 tokens the kernel keeps the keys in shared memory)
            tok = rng.integers(-1, 18, size=T).astype(np.int32)
            perm, so, ids = tbl.segment_tokens(torch.from_numpy(tok).cuda())
            torch.cuda.synchronize()
            rp, ro, rs, _ = oracle.segment(tok, 18)
            assert np.array_equal(perm.cpu().numpy(), rp)
            so, ids = so.cpu().numpy(), ids.cpu().numpy()
            assert ids.tolist() == list(range(18)) + [-1]
            lens = np.diff(so)
            keep = lens > 0
            assert np.array_equal(ids[keep], rs) and np.array_equal(np.concatenate([[0], np.cumsum(lens[keep])]), ro)
        # a retired slot and an out-of-range id go to the -1 group and raise the flag
        tbl.retire_version(3, 1)
        tok = np.array([3, 0, 99, -1, 3], np.int32)
        perm, so, ids = tbl.segment_tokens(torch.from_numpy(tok).cuda())
        assert tbl.device_status() & 1
        assert perm.cpu().numpy().tolist() == [1, 0, 2, 3, 4]
    finally:
        tbl.close()


def test_device_detected_errors_degrade_to_base_output():
    from paper_2608_15241_b200 import binding
    for T in (8, 300):
        w = wl.ragged(T=T, d_in=256, d_out=320, ranks=(8, 16, 4))
        w.seg_offsets = np.array([0, T // 3, 2 * T // 3, T], np.int32)
        w.seg_entry = np.array([0, 1, 2], np.int32)
        site = Site(w, max_slots=4)
        try:
            good, _ = site.run()
            base = oracle.forward(w.x, w.W0, [], [0, T], [-1])[0]
            # unknown slot id in one segment: that segment base-only, flag raised, others intact
            y, flags = site.run(raw_slot_ids=[site.slots[0], 3, site.slots[2]])
            assert flags & binding.FLAG_BAD_SLOT
            a, b = w.seg_offsets[1], w.seg_offsets[2]
            assert oracle.compare(y, base, rows=np.arange(a, b))["ok"]
            assert np.array_equal(y[:a], good[:a]) and np.array_equal(y[b:], good[b:])
            # malformed offsets: base only everywhere
            y, flags = site.run(seg_offsets=[0, 2 * T // 3, T // 3, T])
            assert flags & binding.FLAG_BAD_OFFSETS
            assert oracle.compare(y, base)["ok"]
            y, flags = site.run()
            assert flags == 0 and np.array_equal(y, good)    # the flag is sticky only until read
        finally:
            site.close()


def test_table_operations():
    from paper_2608_15241_b200 import binding
    from paper_2608_15241_b200.binding import Table
    import torch
    tbl = Table(64, 128, max_slots=2)
    try:
        A = torch.zeros((4, 64), dtype=torch.bfloat16, device="cuda")
        B = torch.zeros((128, 4), dtype=torch.bfloat16, device="cuda")
        s0 = tbl.register_adapter(5, 1, A, B, 0.5)
        s1 = tbl.register_adapter(5, 2, A, B, 0.25)
        assert (s0, s1) == (0, 1) and tbl.lookup(5, 2) == 1 and tbl.slot_info(1) == (5, 2, 4, 0.25)
        with pytest.raises(binding.LmlError) as e:
            tbl.register_adapter(5, 2, A, B, 1.0)
        assert e.value.status == 4                               # duplicate
        with pytest.raises(binding.LmlError) as e:
            tbl.register_adapter(6, 1, A, B, 1.0)
        assert e.value.status == 3 and tbl.lookup(5, 1) == 0     # full, unchanged
        with pytest.raises(binding.LmlError) as e:
            binding.register_adapter(tbl.handle, 9, 9, A.data_ptr(), B.data_ptr(), 65, 1.0)
        assert e.value.status == 1                               # rank out of range
        tbl.retire_version(5, 1)
        with pytest.raises(binding.LmlError) as e:
            tbl.lookup(5, 1)
        assert e.value.status == 5
        with pytest.raises(binding.LmlError):
            tbl.retire_version(5, 1)
        assert tbl.register_adapter(6, 1, A, B, 1.0) == 0 and tbl.lookup(5, 2) == 1
        # workspace too small is refused before any launch
        x = torch.zeros((32, 64), dtype=torch.bfloat16, device="cuda")
        W0 = torch.zeros((128, 64), dtype=torch.bfloat16, device="cuda")
        so = torch.tensor([0, 32], dtype=torch.int32, device="cuda")
        ids = torch.tensor([0], dtype=torch.int32, device="cuda")
        small = torch.empty(1024, dtype=torch.uint8, device="cuda")
        with pytest.raises(binding.LmlError) as e:
            tbl.lora_mixed_linear(x, W0, so, ids, workspace=small)
        assert e.value.status == 9
    finally:
        tbl.close()


def test_host_buffer_entry_point():
    import torch
    for w in (wl.ragged(T=300, d_in=256, d_out=320), wl.ragged(T=9, d_in=256, d_out=320, shuffled=True)):
        site = Site(w)
        try:
            ref_y, _ = site.run()
            xh = torch.from_numpy(w.x.view(np.int16)).view(torch.bfloat16).pin_memory()
            yh = torch.empty((w.T, w.d_out), dtype=torch.bfloat16).pin_memory()
            so = torch.from_numpy(w.seg_offsets).pin_memory()
            ids = torch.from_numpy(site.slot_ids()).pin_memory()
            pm = None if w.perm is None else torch.from_numpy(w.perm).pin_memory()
            site.table.lora_mixed_linear_host(xh, site.W0, so, ids, yh, perm_host=pm)
            torch.cuda.synchronize()
            assert np.array_equal(to_bits(yh), ref_y)
            # pageable buffers (for up to 16 tokens the pinned form above takes no copies at all: a kernel
            # reads the inputs from host memory and y is written straight into the caller's buffer)
            xp = torch.from_numpy(w.x.view(np.int16).copy()).view(torch.bfloat16)
            yp = torch.zeros((w.T, w.d_out), dtype=torch.bfloat16)
            pmp = None if w.perm is None else torch.from_numpy(w.perm.copy())
            site.table.lora_mixed_linear_host(xp, site.W0, torch.from_numpy(w.seg_offsets.copy()),
                                              torch.from_numpy(site.slot_ids().copy()), yp, perm_host=pmp)
            torch.cuda.synchronize()
            assert np.array_equal(to_bits(yp), ref_y)
            # twice in a row on the same pinned buffers, then a base-only call
            yh.zero_()
            site.table.lora_mixed_linear_host(xh, site.W0, so, ids, yh, perm_host=pm)
            site.table.lora_mixed_linear_host(xh, site.W0, so, ids, yh, perm_host=pm)
            torch.cuda.synchronize()
            assert np.array_equal(to_bits(yh), ref_y)
        finally:
            site.close()


@pytest.mark.parametrize("kw", [dict(T=2100, d_in=256, d_out=520), dict(T=2048, d_in=520, d_out=264),
                                dict(T=4000, d_in=264, d_out=1000)])
def test_host_buffer_call_in_chunks(kw):
    """Large calls (2048 tokens and more) on pinned buffers run in eight chunks of whole row tiles with the copies on the table's own
    streams.  Same results as the device-buffer call (up to the order of the split-K sums where a chunk is
    small enough for that kernel), the oracle within tolerance, malformed offsets caught for the whole
    call, and back-to-back calls on the same buffers stay ordered."""
    import torch
    from paper_2608_15241_b200 import binding
    w = wl.ragged(ranks=(4, 16, 1, 33, 64), **kw)
    site = Site(w)
    try:
        ref_y, _ = site.run()
        xh = torch.from_numpy(w.x.view(np.int16)).view(torch.bfloat16).pin_memory()
        yh = torch.zeros((w.T, w.d_out), dtype=torch.bfloat16).pin_memory()
        so = torch.from_numpy(w.seg_offsets).pin_memory()
        ids = torch.from_numpy(site.slot_ids()).pin_memory()
        for _ in range(3):
            site.table.lora_mixed_linear_host(xh, site.W0, so, ids, yh)
        torch.cuda.synchronize()
        assert site.table.device_status() == 0
        got = to_bits(yh)
        ref, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, w.seg_entry, None)
        assert oracle.compare(got, ref)["ok"]
        diff = np.abs(wl.bf16_bits_to_f64(got) - wl.bf16_bits_to_f64(ref_y))
        assert (diff <= 2.0 ** -7 * np.maximum(1.0, np.abs(wl.bf16_bits_to_f64(ref_y)))).all()
        # no adapters at all
        yh.zero_()
        site.table.lora_mixed_linear_host(xh, site.W0, None, None, yh)
        torch.cuda.synchronize()
        base = oracle.forward(w.x, w.W0, [], [0, w.T], [-1])[0]
        assert oracle.compare(to_bits(yh), base)["ok"]
        # malformed offsets: base output everywhere, flag raised
        bad = w.seg_offsets.copy()
        bad[1], bad[2] = bad[2], bad[1]
        if bad[1] != bad[2]:
            site.table.lora_mixed_linear_host(xh, site.W0, torch.from_numpy(bad).pin_memory(), ids, yh)
            torch.cuda.synchronize()
            assert site.table.device_status() & binding.FLAG_BAD_OFFSETS
            assert oracle.compare(to_bits(yh), base)["ok"]
    finally:
        site.close()


@pytest.mark.parametrize("T,G", [(16, 200), (7, 129), (16, 128)])
def test_decode_with_many_mostly_empty_segments(T, G):
    """More segments than the decode kernel caches in shared memory (128): the lookup then searches
    the arrays in global memory.  Most segments are empty and may repeat slots."""
    w = wl.ragged(T=T, d_in=520, d_out=264, ranks=(4, 16, 1, 33, 64))
    rng = np.random.default_rng(G * 31 + T)
    cuts = np.sort(rng.integers(0, T + 1, size=G - 1))
    so = np.concatenate([[0], cuts, [T]]).astype(np.int32)
    se = rng.integers(-1, len(w.entries), size=G).astype(np.int32)
    site = Site(w)
    y, flags = site.run(seg_offsets=so, seg_entry=se, perm=None)
    ref, _ = oracle.forward(w.x, w.W0, w.entries, so, se)
    r = oracle.compare(y, ref)
    assert flags == 0 and r["ok"], r
    site.close()
