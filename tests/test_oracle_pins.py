"""Pins for the fp64 CPU oracle: each test fixes it against something other than itself —
the definition's invariants, closed forms, numpy's float64 matmul, a hand-worked example,
and a brute-force twin with a different loop nest."""
import os

import numpy as np
import pytest

import oracle
from paper_2608_15241_b200 import workloads as wl

GOLDEN = os.path.join(os.path.dirname(__file__), "golden")


def bits(a):
    return wl.f32_to_bf16_bits(np.asarray(a, dtype=np.float32))


def f64(b):
    return wl.bf16_bits_to_f64(b)


def entry(A, B, scale, aid=0, ver=1):
    A = np.atleast_2d(np.asarray(A, dtype=np.float32))
    B = np.atleast_2d(np.asarray(B, dtype=np.float32))
    return wl.AdapterEntry(aid, ver, A.shape[0], float(scale), bits(A), bits(B))


def numpy_reference(w):
    """Independent statement with numpy float64 matmul (a library routine, not the oracle's
    loops): per segment y = x W0^T + s (x A^T) B^T."""
    x, W0 = f64(w.x), f64(w.W0)
    y = np.zeros((w.T, w.d_out))
    for g in range(w.G):
        pos = np.arange(w.seg_offsets[g], w.seg_offsets[g + 1])
        rows = pos if w.perm is None else w.perm[pos]
        yy = x[rows] @ W0.T
        e = int(w.seg_entry[g])
        if e >= 0:
            ent = w.entries[e]
            yy = yy + float(np.float32(ent.scale)) * ((x[rows] @ f64(ent.A).T) @ f64(ent.B).T)
        y[rows] = yy
    return y


def parse_golden(path):
    out = {}
    for line in open(path):
        line = line.strip()
        if not line or line.startswith("#"):
            continue
        k, v = line.split("=", 1)
        rows = [[float(t) for t in r.split()] for r in v.split(";")]
        out[k.strip()] = np.array(rows, dtype=np.float64)
    return out


def test_hand_worked_example():
    g = parse_golden(os.path.join(GOLDEN, "hand_worked_2x2.txt"))
    x, W0 = bits(g["x"]), bits(g["W0"])
    ent = [entry(g["A"], g["B"], g["scale"][0, 0])]
    y, fl = oracle.forward(x, W0, ent, [0, 2], [0])
    assert fl == 0 and np.array_equal(y, g["y_both_rows_on_adapter"])
    y, _ = oracle.forward(x, W0, ent, [0, 1, 2], [0, -1])
    assert np.array_equal(y, g["y_row1_without_adapter"])
    y, _ = oracle.forward(x, W0, ent, [0, 2], [-1])
    assert np.array_equal(y, g["y_no_adapter"])
    # B is [N][r]: swapping its two entries must swap the deltas (catches a transposed B)
    ent2 = [entry(g["A"], g["B"][::-1].copy(), g["scale"][0, 0])]
    y, _ = oracle.forward(x, W0, ent2, [0, 2], [0])
    assert np.array_equal(y, np.array([[2.5 + 0.25, -1.5 - 1.0], [0.5 - 1.0, -6.25 + 4.0]]))


def test_zero_B_is_exactly_base():
    w = wl.tiny()
    base, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, np.full(w.G, -1, np.int32))
    for e in w.entries:
        e.B = np.zeros_like(e.B)
    y, fl = oracle.forward_workload(w)
    assert fl == 0 and np.array_equal(y, base)


def test_single_slot_equals_merged_weight():
    w = wl.tiny()
    ent = w.entries[1]
    y, _ = oracle.forward(w.x, w.W0, w.entries, [0, w.T], [1])
    merged = f64(w.W0) + float(np.float32(ent.scale)) * (f64(ent.B) @ f64(ent.A))  # [N][K], unrounded
    ref = f64(w.x) @ merged.T
    assert np.abs(y - ref).max() <= 1e-12 * np.abs(ref).max()
    # and the LoRA term is not negligible in this check
    base = f64(w.x) @ f64(w.W0).T
    assert np.abs(ref - base).max() > 1e-3


def test_segment_permutation_permutes_rows_exactly():
    w = wl.tiny()
    y, _ = oracle.forward_workload(w)
    # reorder segments (2, 0, 1) together with their rows
    order = [2, 0, 1]
    lens = np.diff(w.seg_offsets)
    rows = np.concatenate([np.arange(w.seg_offsets[g], w.seg_offsets[g + 1]) for g in order])
    off = np.concatenate([[0], np.cumsum(lens[order])]).astype(np.int32)
    y2, _ = oracle.forward(w.x[rows], w.W0, w.entries, off, w.seg_entry[order])
    assert np.array_equal(y2, y[rows])


def test_no_adapter_rows_are_base_only_and_others_unchanged():
    w = wl.tiny()
    y, _ = oracle.forward_workload(w)
    base, _ = oracle.forward(w.x, w.W0, [], [0, w.T], [-1])
    se = w.seg_entry.copy()
    se[1] = -1
    y2, _ = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, se)
    a, b = w.seg_offsets[1], w.seg_offsets[2]
    assert np.array_equal(y2[a:b], base[a:b])
    assert np.array_equal(y2[:a], y[:a]) and np.array_equal(y2[b:], y[b:])
    assert not np.array_equal(y[a:b], base[a:b])


@pytest.mark.parametrize("maker", [wl.tiny, lambda: wl.ragged(T=37, d_in=40, d_out=24, ranks=(4, 3, 1, 8, 5)),
                                   lambda: wl.ragged(T=37, d_in=40, d_out=24, ranks=(4, 3, 1, 8, 5), shuffled=True)])
def test_brute_force_twin_and_numpy_agree(maker):
    w = maker()
    y, fl = oracle.forward_workload(w)
    assert fl == 0
    yb = oracle.forward_brute(w.x, w.W0, w.entries, w.seg_offsets, w.seg_entry, w.perm)
    ref = numpy_reference(w)
    scale = np.abs(ref).max()
    assert np.abs(y - yb).max() <= 1e-12 * scale
    assert np.abs(y - ref).max() <= 1e-12 * scale


def test_base_term_matches_numpy_float64():
    w = wl.ragged(T=50, d_in=136, d_out=72)
    y, _ = oracle.forward(w.x, w.W0, [], [0, w.T], [-1])
    ref = f64(w.x) @ f64(w.W0).T
    assert np.abs(y - ref).max() <= 1e-13 * np.abs(ref).max()


def test_one_hot_input_reads_one_weight_column():
    K, N, r = 24, 16, 3
    W0 = wl.normal_bf16(5, 1, (N, K), 0.5)
    A = wl.normal_bf16(5, 2, (r, K), 0.5)
    B = wl.normal_bf16(5, 3, (N, r), 0.5)
    ent = [wl.AdapterEntry(0, 1, r, 0.75, A, B)]
    x = np.zeros((K, K), dtype=np.float32)
    x[np.arange(K), np.arange(K)] = 1.0
    y, _ = oracle.forward(bits(x), W0, ent, [0, K], [0])
    for k in range(K):
        expect = f64(W0)[:, k] + 0.75 * (f64(B) @ f64(A)[:, k])
        assert np.abs(y[k] - expect).max() <= 1e-15


def test_constant_inputs_closed_form():
    # x = 1, W0 = c, A = 1, B = 1  =>  y = K*c + s*r*K for every element
    K, N, T, r, s, c = 64, 8, 3, 5, 0.25, 0.5
    x = bits(np.ones((T, K)))
    W0 = bits(np.full((N, K), c))
    ent = [entry(np.ones((r, K)), np.ones((N, r)), s)]
    y, _ = oracle.forward(x, W0, ent, [0, T], [0])
    assert np.all(y == K * c + s * r * K)
    # distinct A rows and B columns: A[j][k] = j+1, B[n][j] = n+1  =>  delta = s*K*(n+1)*sum(j+1)
    A = np.repeat(np.arange(1, r + 1, dtype=np.float32)[:, None], K, axis=1)
    B = np.repeat(np.arange(1, N + 1, dtype=np.float32)[:, None], r, axis=1)
    y, _ = oracle.forward(x, W0, [entry(A, B, s)], [0, T], [0])
    expect = K * c + s * K * np.arange(1, N + 1) * (r * (r + 1) / 2)
    assert np.array_equal(y, np.tile(expect, (T, 1)))


def test_integer_lattice_is_integral_and_matches_numpy_exactly():
    w = wl.lattice()
    y, fl = oracle.forward_workload(w)
    assert fl == 0
    assert np.array_equal(y, np.round(y)) and np.abs(y).max() <= 80
    assert np.array_equal(y, numpy_reference(w))
    # the outputs are exactly representable in bf16
    assert np.array_equal(f64(bits(y)), y)


def test_version_routing_opposite_B():
    K, N, r, T = 32, 16, 4, 10
    x = wl.normal_bf16(3, 1, (T, K), 1.0)
    W0 = wl.normal_bf16(3, 2, (N, K), 0.1)
    A = wl.normal_bf16(3, 3, (r, K), 0.1)
    B = wl.normal_bf16(3, 4, (N, r), 0.1)
    Bneg = (B ^ np.uint16(0x8000)).astype(np.uint16)  # exact negation in bf16
    ents = [wl.AdapterEntry(0, 1, r, 1.5, A, B), wl.AdapterEntry(0, 2, r, 1.5, A, Bneg),
            wl.AdapterEntry(1, 1, r, 1.5, wl.normal_bf16(3, 5, (r, K), 0.1), B)]
    base, _ = oracle.forward(x, W0, [], [0, T], [-1])
    y_old, _ = oracle.forward(x, W0, ents, [0, T], [0])
    y_new, _ = oracle.forward(x, W0, ents, [0, T], [1])
    assert np.abs((y_old - base) + (y_new - base)).max() <= 1e-15
    # mixed call: first half old, second half new; resident-but-unbound entry 2 changes nothing
    y_mix, _ = oracle.forward(x, W0, ents, [0, 5, T], [0, 1])
    assert np.array_equal(y_mix[:5], y_old[:5]) and np.array_equal(y_mix[5:], y_new[5:])
    y_mix2, _ = oracle.forward(x, W0, ents[:2], [0, 5, T], [0, 1])
    assert np.array_equal(y_mix, y_mix2)


def test_perm_addresses_rows():
    w = wl.ragged(T=41, d_in=48, d_out=40, ranks=(4, 2, 6, 8, 5), shuffled=True)
    y, _ = oracle.forward_workload(w)
    # same call with rows physically gathered and no perm
    yg, _ = oracle.forward(w.x[w.perm], w.W0, w.entries, w.seg_offsets, w.seg_entry)
    assert np.array_equal(y[w.perm], yg)
    # per-row binding agrees with token_entry
    for p in range(w.T):
        g = np.searchsorted(w.seg_offsets, p, side="right") - 1
        while w.seg_offsets[g + 1] <= p:
            g += 1
        assert w.token_entry[w.perm[p]] == w.seg_entry[g]


def test_positions_subset_matches_full():
    w = wl.ragged()
    y, _ = oracle.forward_workload(w)
    pos = np.array([0, 5, 77, 200, w.T - 1], dtype=np.int32)
    ys, _ = oracle.forward_workload(w, positions=pos)
    assert np.array_equal(ys[pos], y[pos])
    mask = np.ones(w.T, bool)
    mask[pos] = False
    assert np.all(ys[mask] == 0)


def test_error_flags():
    w = wl.tiny()
    base, _ = oracle.forward(w.x, w.W0, [], [0, w.T], [-1])
    good, _ = oracle.forward_workload(w)
    # unknown entry id: that segment gets base only, others unaffected
    se = w.seg_entry.copy()
    se[0] = 7
    y, fl = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, se)
    assert fl & oracle.FLAG_BAD_SLOT
    a = w.seg_offsets[1]
    assert np.array_equal(y[:a], base[:a]) and np.array_equal(y[a:], good[a:])
    # dead entry behaves the same way
    y, fl = oracle.forward(w.x, w.W0, w.entries, w.seg_offsets, w.seg_entry, live=[1, 0, 1])
    assert fl & oracle.FLAG_BAD_SLOT
    a, b = w.seg_offsets[1], w.seg_offsets[2]
    assert np.array_equal(y[a:b], base[a:b]) and np.array_equal(y[:a], good[:a])
    # malformed offsets: base only everywhere
    y, fl = oracle.forward(w.x, w.W0, w.entries, [0, 40, 30, w.T], w.seg_entry)
    assert fl & oracle.FLAG_BAD_OFFSETS and np.array_equal(y, base)
    y, fl = oracle.forward(w.x, w.W0, w.entries, [0, 30, 50, w.T - 1], w.seg_entry)
    assert fl & oracle.FLAG_BAD_OFFSETS and np.array_equal(y, base)


def test_empty_inputs():
    w = wl.tiny()
    y, fl = oracle.forward(w.x[:0], w.W0, w.entries, [0], [])
    assert y.shape == (0, w.d_out) and fl == 0
    y, fl = oracle.forward(w.x, w.W0, w.entries, [0], [])  # G = 0: base only
    base, _ = oracle.forward(w.x, w.W0, [], [0, w.T], [-1])
    assert np.array_equal(y, base)


def test_segmentation_reference_against_sorted():
    rng = np.random.default_rng(0)
    for T, S in [(0, 3), (1, 1), (64, 3), (500, 18), (257, 64)]:
        te = rng.integers(-1, S, size=T).astype(np.int32)
        perm, off, se, fl = oracle.segment(te, S)
        assert fl == 0
        # python's sorted() is stable: an independent statement of the rule
        expect = sorted(range(T), key=lambda t: (S if te[t] < 0 else te[t]))
        assert perm.tolist() == expect
        assert off[0] == 0 and off[-1] == T and np.all(np.diff(off) > 0)
        for g in range(len(se)):
            assert np.all(te[perm[off[g]:off[g + 1]]] == se[g])
        keys = [S if s < 0 else s for s in se]
        assert keys == sorted(set(S if v < 0 else v for v in te.tolist()))
        p2, o2, s2 = wl.group_tokens(te, S)
        assert np.array_equal(p2, perm) and np.array_equal(o2, off) and np.array_equal(s2, se)
    perm, off, se, fl = oracle.segment(np.array([0, 9, -5, 1], np.int32), 2)
    assert fl & oracle.FLAG_BAD_SLOT and perm.tolist() == [0, 3, 1, 2] and se.tolist() == [0, 1, -1]


def test_compare_criterion():
    o = np.array([[0.5, -200.0, 3.0]])
    ok = bits(np.array([[0.5078125, -201.0, 3.0]]))  # within 1e-2*max(1,|o|)
    assert oracle.compare(ok, o)["ok"]
    bad = bits(np.array([[0.515625, -200.0, 3.0]]))  # 0.0156 > 1e-2
    assert not oracle.compare(bad, o)["ok"]
    # Frobenius criterion alone can fail: many small errors each inside the element bound
    o2 = np.full((1, 1000), 1.0)
    g2 = bits(np.full((1, 1000), 1.0078125))
    r = oracle.compare(g2, o2)
    assert r["worst_tol_ratio"] <= 1.0 and r["rel_fro"] > 5e-3 and not r["ok"]
