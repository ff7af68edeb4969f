"""The seeded input recipes produce the shapes and structure the workloads are defined by."""
import numpy as np

from paper_2608_15241_b200 import workloads as wl


def test_bf16_rounding_is_nearest_even():
    f = np.array([1.0, 1.00390625, 1.01171875, -3.0e-3, 0.0], dtype=np.float32)
    b = wl.f32_to_bf16_bits(f)
    back = wl.bf16_bits_to_f64(b)
    # 1 + 2^-8 is a tie between 1.0 and 1 + 2^-7: goes to the even mantissa (1.0);
    # 1 + 3*2^-8 is a tie between 1 + 2^-7 and 1 + 2^-6: goes to 1 + 2^-6
    assert back[0] == 1.0 and back[1] == 1.0 and back[2] == 1.015625 and back[4] == 0.0
    assert abs(back[3] - f[3]) <= abs(f[3]) * 2.0 ** -8


def test_streams_are_independent_and_seeded():
    a = wl.normal_bf16(0, 1, (64, 64), 1.0)
    assert np.array_equal(a, wl.normal_bf16(0, 1, (64, 64), 1.0))
    assert not np.array_equal(a, wl.normal_bf16(1, 1, (64, 64), 1.0))
    assert not np.array_equal(a, wl.normal_bf16(0, 2, (64, 64), 1.0))
    v = wl.bf16_bits_to_f64(wl.normal_bf16(0, 2, (512, 512), 0.02))
    assert abs(v.std() - 0.02) < 5e-4 and abs(v.mean()) < 2e-4


def test_tiny_config():
    w = wl.tiny()
    assert (w.d_in, w.d_out, w.T) == (256, 256, 64)
    assert w.seg_offsets.tolist() == [0, 30, 50, 64] and w.seg_entry.tolist() == [0, 1, 2]
    assert [e.rank for e in w.entries] == [4, 8, 8]
    assert [e.scale for e in w.entries] == [0.5, 0.25, 0.25]
    assert abs(w.flops() - (2 * 64 * 256 * 256 + 2 * 512 * (30 * 4 + 20 * 8 + 14 * 8))) < 1


def test_decode_config():
    w = wl.decode_q_proj()
    assert (w.d_in, w.d_out, w.T, len(w.entries)) == (4096, 4096, 8, 5)
    assert w.seg_entry.tolist() == [0, 1, 2, 3]
    assert (w.entries[0].adapter_id, w.entries[0].version) == (0, 1)
    assert (w.entries[4].adapter_id, w.entries[4].version) == (0, 2)
    assert not np.array_equal(w.entries[0].A, w.entries[4].A)
    assert abs(w.bytes() - 34.73e6) < 0.02e6  # 4 used entries, the resident unused one counts 0
    assert wl.decode_q_proj(split_versions=True).seg_entry.tolist() == [0, 4, 1, 2, 3]


def test_prefill_config():
    w = wl.prefill_q_proj()
    assert np.diff(w.seg_offsets).tolist() == [1024, 512, 384, 128]
    assert (w.entries[0].adapter_id, w.entries[0].version) == (0, 2)
    assert (w.entries[4].adapter_id, w.entries[4].version) == (0, 1)
    assert 4 not in w.seg_entry.tolist()
    assert abs(w.flops() - (68.72e9 + 0.54e9)) < 0.01e9


def test_mlp_config_structure():
    w = wl.mlp_up_gate(T=512, d_in=64, d_out=96)
    assert (w.token_entry == -1).sum() == 51 and w.seg_entry[-1] == -1
    assert np.all(np.diff(w.seg_offsets) > 0) and w.seg_offsets[-1] == 512
    lens = np.diff(w.seg_offsets)[:-1]
    assert lens[0] == lens.max()  # Zipf: entry 0 is the most popular
    ws = wl.mlp_up_gate(T=512, d_in=64, d_out=96, shuffled=True)
    assert sorted(ws.perm.tolist()) == list(range(512))
    assert np.array_equal(np.diff(ws.seg_offsets), np.diff(w.seg_offsets))
    for g in range(ws.G):
        rows = ws.perm[ws.seg_offsets[g]:ws.seg_offsets[g + 1]]
        assert np.all(ws.token_entry[rows] == ws.seg_entry[g])
        assert np.all(np.diff(rows) > 0)  # stable grouping


def test_sweep_cell():
    w = wl.layer_sweep("q", 128)
    assert len(w.entries) == 18 and w.T == 128 and (w.d_in, w.d_out) == (4096, 4096)
    assert {(e.adapter_id, e.version) for e in w.entries} >= {(0, 1), (0, 2), (1, 1), (1, 2)}
    assert set(w.seg_entry.tolist()) >= {0, 16}  # both versions of the most popular adapter serve
    assert wl.LAYER_PROJECTIONS["down"] == (11008, 4096)


def test_lattice_and_ragged_structure():
    w = wl.lattice()
    x = wl.bf16_bits_to_f64(w.x)
    assert np.all((x != 0).sum(axis=1) == 16) and set(np.unique(x)) <= {-1.0, 0.0, 1.0}
    assert 0 in np.diff(w.seg_offsets) and -1 in w.seg_entry
    r = wl.ragged()
    assert r.seg_offsets[0] == 0 and r.seg_offsets[-1] == r.T and np.all(np.diff(r.seg_offsets) >= 0)
    assert len(set(r.seg_entry.tolist())) < r.G  # some entry serves two segments
